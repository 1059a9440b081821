#!/usr/bin/env python
"""Benchmark of the PWLQ hot path on B200.

One step = one pass of the whole path over one batch of synthetic tensors:
abs-max -> K-candidate breakpoint search -> quantize (packed codes + region mask) -> dequantize.
The headline workload is the full set of ResNet-50 v1.5 conv + fc weight shapes quantized per
output channel at 4 bits with K = 256 candidates (27 560 rows, 25.5 M values, 6.53 G
value-candidate evaluations per step).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

Prints ONE JSON line.
  value          value-candidate evaluations per second of the whole step, inputs resident in HBM
  e2e            the same through the host-buffer entry point, host<->device copies timed
  roofline       the search kernels against the FP32 pipe: `frac` counts the 6 lane-operations
                 the definition has per evaluation, `frac_issued` the 4 (center) or 5 (tail) the
                 kernel issues; `peak` is derived from the data sheet, `peak_measured` comes from
                 a packed-FMA micro-benchmark run here
  hbm_stages     the three HBM-bound kernels as timed inside the step (one cold launch each after
                 the L2 eviction); hbm_streaming: the same kernels back to back on the workload's
                 rows repeated until they exceed L2, and under `mapped` the same calls given row
                 maps built once per layout (pwlq_rowmap_build) where several rows share a span
  sustained      at least two seconds of back-to-back steps with the SM clock sampled meanwhile
  workloads      the other benchmark configurations, each with its stage times and fractions
  extras         the calls beyond the four-call path (two / three breakpoints, analytic selection,
                 bias correction, dense packing) as single cold launches
  cpu_baseline   the CPU oracle on the host cores (all cores, and one thread)
With N > 1 (torchrun) every rank processes its own batch (rows are independent: no collective on
the data path) and the slowest rank's time counts.  `--impl reference` times the CPU oracle on a
bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import ctypes
import json
import os
import statistics
import subprocess
import sys
import threading
import time
from concurrent.futures import ThreadPoolExecutor

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2002_00104_b200 import workloads as W  # noqa: E402

METRIC = "pwlq_search_quantize_throughput"
UNIT = "Gelem*cand/s"
SM_COUNT, FP32_LANES_PER_SM, SM_MAX_GHZ = 148, 128, 1.965
ALU_PEAK_TLANEOPS = SM_COUNT * FP32_LANES_PER_SM * SM_MAX_GHZ / 1e3     # 37.2 T lane-ops/s
LANE_OPS_PER_ELEM_CAND = 6      # sub, mul, 2 adds (round to nearest even), fma, fma
L2_FLUSH_BYTES = 256 << 20
L2_BYTES = 126 << 20

WORKLOADS = {
    "resnet50": W.resnet50,
    "single_conv": W.single_conv,
    "mobilenetv2": W.mobilenetv2,
    "relu_activation": W.relu_activation,
    "laplace4096": W.laplace_matrix,
}


def make_workload(args, seed, name=None):
    """The named workload; --bits / --K / --rows / --cols override its defaults (sweeps)."""
    name = name or args.workload
    kw = {} if seed is None else {"seed": seed}
    if name == "laplace4096" and name == args.workload:
        if args.rows: kw["rows"] = args.rows
        if args.cols: kw["cols"] = args.cols
    w = WORKLOADS[name](**kw)
    if name == args.workload:
        if args.bits: w.bits = args.bits
        if args.K: w.K = args.K
    return w


def config_of(w: W.Workload, scheme: str, world: int):
    """The `config` object; both arms (--impl ours / reference) print the same one."""
    return {"workload": w.name, "bits": w.bits, "K": w.K, "rows": w.C, "values": w.total,
            "elem_cand_per_step": w.elem_cand, "code_layout": "packed", "scheme": scheme,
            "l2": f"flushed between steps by writing {L2_FLUSH_BYTES >> 20} MiB",
            "parallelism": f"independent batches x{world}"}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": 6650.0}, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while a timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc, self.thread = index, [], None, None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            return self
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        self.thread.join(timeout=2)
        sm, mx, power, reasons = [], [], [], set()
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1])); power.append(float(r[2]))
            except (ValueError, IndexError):
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                "sw_power_cap"), r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        busy = [s for s in sm if s > 0]
        return {"sm_mhz": statistics.median(busy) if busy else None,
                "sm_max_mhz": max(mx) if mx else None, "reasons": sorted(reasons),
                "samples": len(busy), "power_w_max": max(power) if power else None}


# --------------------------------------------------------------------------- CPU oracle timing
def oracle_sample(w: W.Workload, budget_evals: float):
    """A stratified subset of rows (every s-th row, so each layer shape is represented in
    proportion) holding about `budget_evals` value-candidate evaluations; for a single row, a
    prefix of its values.  Returns (values, row_offsets, description)."""
    if w.C == 1:
        n = max(1, min(w.total, int(budget_evals // w.K)))
        return (w.x[:n], np.array([0, n], np.int64),
                f"first {n} of {w.total} values of the single row, all {w.K} candidates")
    stride = max(1, int(round(w.elem_cand / budget_evals)))
    rows = np.arange(0, w.C, stride)
    lens = np.diff(w.row_offsets)[rows]
    xs = np.concatenate([w.x[w.row_offsets[c]:w.row_offsets[c + 1]] for c in rows])
    ro = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    return xs, ro, f"every {stride}th row ({rows.size} of {w.C} rows), all {w.K} candidates"


def time_oracle(w: W.Workload, xs, ro, threads: int):
    """Times oracle abs-max + search + quantize + dequantize over the sample.  The oracle is
    single-threaded C; with threads > 1 the sample's rows are cut into `threads` contiguous groups
    of about equal size and every host thread makes ONE ragged oracle call per stage on its group
    (a single row is cut over the candidates for the search instead)."""
    import oracle
    oracle.build()
    ratios = W.ratio_grid(w.K)
    C = ro.size - 1

    def rows_job(r0, r1):
        b, e = int(ro[r0]), int(ro[r1])
        x, o = xs[b:e], (ro[r0:r1 + 1] - ro[r0]).astype(np.int64)
        m = oracle.absmax(x, o)
        r = oracle.search(x, w.bits, ratios, m=m, row_offsets=o, want_sse=False)
        codes, mask, _ = oracle.quantize(x, w.bits, m, r["p"], layout=1, row_offsets=o,
                                         want_fake=False)
        oracle.dequantize(codes, mask, w.bits, m, r["p"], layout=1, row_offsets=o)

    t0 = time.perf_counter()
    if C == 1:
        m = oracle.absmax(xs)
        chunks = [c for c in np.array_split(np.arange(w.K), threads) if c.size]
        with ThreadPoolExecutor(threads) as ex:
            parts = list(ex.map(lambda ks: oracle.search(xs, w.bits, ratios[ks], m=m)["sse64"][0],
                                chunks))
        p = np.array([m[0] * ratios[int(np.argmin(np.concatenate(parts)))]], np.float32)
        codes, mask, _ = oracle.quantize(xs, w.bits, m, p, layout=1, want_fake=False)
        oracle.dequantize(codes, mask, w.bits, m, p, C=1, n=xs.size, layout=1)
    elif threads > 1:
        targets = [int(ro[-1]) * k // threads for k in range(1, threads)]
        cuts = [0] + [int(np.searchsorted(ro, t)) for t in targets] + [C]
        jobs = [(a, b) for a, b in zip(cuts, cuts[1:]) if b > a]
        with ThreadPoolExecutor(threads) as ex:
            list(ex.map(lambda j: rows_job(*j), jobs))
    else:
        rows_job(0, C)
    dt = time.perf_counter() - t0
    return int(ro[-1]) * w.K, dt


def cpu_baseline_of(w: W.Workload, seconds: float = 12.0):
    """All-cores and single-thread oracle figures on bounded samples of the workload."""
    cores = os.cpu_count() or 1
    xs, ro, _ = oracle_sample(w, 2e8)                           # short calibration
    ev, dt = time_oracle(w, xs, ro, cores)
    xs, ro, what = oracle_sample(w, min(w.elem_cand, seconds * ev / dt))
    ev, dt, passes = 0, 0.0, 0
    while dt < 0.7 * seconds and passes < 8:                    # repeated if the box is faster
        e1, d1 = time_oracle(w, xs, ro, cores)
        ev += e1; dt += d1; passes += 1
    out = {"value": ev / dt / 1e9, "unit": UNIT, "cores": cores, "kind": "oracle",
           "sample": what + f", {passes} pass(es)", "seconds": dt}
    xs1, ro1, what1 = oracle_sample(w, min(w.elem_cand, 4.0 * ev / dt / cores))   # about 4 s
    e1, d1 = time_oracle(w, xs1, ro1, 1)
    out["single_thread"] = {"value": e1 / d1 / 1e9, "unit": UNIT, "cores": 1, "sample": what1,
                            "seconds": d1}
    return out


def run_reference(args, rank, world):
    if rank != 0:
        return
    w = make_workload(args, None)
    cores = os.cpu_count() or 1
    # size the per-step sample from a short calibration so that the run ends within minutes
    xs, ro, _ = oracle_sample(w, 2e8)
    ev, dt = time_oracle(w, xs, ro, cores)
    rate = ev / dt
    per_step = min(w.elem_cand, rate * max(2.0, 90.0 / max(1, args.steps + args.warmup)))
    xs, ro, what = oracle_sample(w, per_step)
    for _ in range(args.warmup):
        time_oracle(w, xs, ro, cores)
    tot_ev, tot_dt = 0, 0.0
    for _ in range(args.steps):
        ev, dt = time_oracle(w, xs, ro, cores)
        tot_ev += ev; tot_dt += dt
    val = tot_ev / tot_dt / 1e9
    line = {"metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * tot_dt / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic", "impl": "reference",
            "config": config_of(w, args.scheme, world),
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": "per step: " + what},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------ GPU arm
def issued_lane_ops(w: W.Workload, max_rows: int = 400):
    """Lane-operations the search kernels issue per evaluation on this workload: 4 for a value in
    a candidate's center piece, 5 in its tail piece (the definition counts 6 for both).  The share
    of center evaluations is counted exactly on a stratified sample of rows."""
    ratios = W.ratio_grid(w.K).astype(np.float64)
    rows = np.unique(np.linspace(0, w.C - 1, min(w.C, max_rows)).astype(np.int64))
    center = evals = 0
    for c in rows:
        a = np.abs(w.x[w.row_offsets[c]:w.row_offsets[c + 1]])
        if a.size > 200000:
            a = a[:: a.size // 200000]
        if a.size == 0:
            continue
        a = np.sort(a)
        p = (np.float32(a[-1]) * W.ratio_grid(w.K)).astype(np.float32)
        center += int(np.searchsorted(a, p, side="right").sum())
        evals += a.size * w.K
    share = center / max(evals, 1)
    return 4.0 * share + 5.0 * (1.0 - share), share, ratios.size


class FP32Peak:
    """The packed-FMA micro-benchmark (libpwlq_peak.so, built from csrc/fp32_peak.cu)."""

    def __init__(self):
        from paper_2002_00104_b200 import build
        build.build()
        self.lib = ctypes.CDLL(build.PEAK_LIB)
        self.lib.pwlq_peak_launch.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                              ctypes.c_void_p, ctypes.c_void_p]

    def run(self, torch, mode: int, ms_target: float = 40.0):
        """T lane-ops/s of one launch of about `ms_target` ms (CUDA events)."""
        blocks = SM_COUNT * 8
        threads = self.lib.pwlq_peak_threads()
        out = torch.empty(blocks * threads, dtype=torch.float32, device="cuda")
        st = torch.cuda.current_stream()
        per_trip = self.lib.pwlq_peak_instr_per_trip() * self.lib.pwlq_peak_lanes(mode)

        def once(iters):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(st)
            rc = self.lib.pwlq_peak_launch(mode, blocks, iters, out.data_ptr(), st.cuda_stream)
            b.record(st)
            torch.cuda.synchronize()
            if rc != 0:
                raise RuntimeError(f"pwlq_peak_launch: CUDA error {rc}")
            return a.elapsed_time(b)

        once(200)
        ms = once(2000)
        iters = max(2000, int(2000 * ms_target / max(ms, 1e-3)))
        ms = min(once(iters), once(iters))
        return blocks * threads * iters * per_trip / (ms * 1e-3) / 1e12


class DevicePath:
    """One workload resident on the device, with everything a step needs."""

    def __init__(self, torch, pwlq, w: W.Workload, dev, scheme="signed"):
        self.torch, self.pwlq, self.w, self.dev = torch, pwlq, w, dev
        self.unsigned = scheme == "unsigned"
        self.layout = pwlq.CODES_PACKED
        self.max_n = int(np.diff(w.row_offsets).max())
        self.dense_n = w.uniform_n()
        x = torch.from_numpy(w.x).to(dev)
        if self.dense_n is not None:
            self.x, self.ro = x.view(w.C, self.dense_n), None
        else:
            self.x, self.ro = x, torch.from_numpy(w.row_offsets).to(dev)
        self.set_grid(w.bits, w.K)
        f32 = lambda n: torch.empty(n, dtype=torch.float32, device=dev)
        self.m, self.lo, self.y = f32(w.C), f32(w.C), f32(w.total)
        self.sout = {"p": f32(w.C), "err": f32(w.C),
                     "idx": torch.empty(w.C, dtype=torch.int32, device=dev), "sse": None}
        self.mask = torch.empty((w.total + 7) // 8, dtype=torch.uint8, device=dev)

    def set_grid(self, bits, K):
        torch, pwlq, w = self.torch, self.pwlq, self.w
        self.bits, self.K = bits, K
        self.ratios_np = W.ratio_grid(K)
        self.ratios = torch.from_numpy(self.ratios_np).to(self.dev)
        self.ws = torch.empty(max(256, pwlq.search_workspace_bytes(w.C, self.max_n, K)),
                              dtype=torch.uint8, device=self.dev)
        self.codes = torch.empty(pwlq.code_bytes(w.total, bits, self.layout), dtype=torch.uint8,
                                 device=self.dev)

    @property
    def elem_cand(self):
        return self.w.total * self.K

    def io_bytes(self):
        """Algorithmic bytes of quantize and of dequantize: values + codes + region bits."""
        return self.w.total * 4 + self.codes.numel() + self.mask.numel()

    def step(self, ev=None):
        """One pass of the whole path; ev = 5 CUDA events to record between the stages."""
        pwlq, w, x, ro, m, lo = self.pwlq, self.w, self.x, self.ro, self.m, self.lo
        st = self.torch.cuda.current_stream()
        if ev: ev[0].record(st)
        if self.unsigned:
            pwlq.minmax(x, row_offsets=ro, out=(lo, m))
            if ev: ev[1].record(st)
            pwlq.search_unsigned(x, self.bits, self.ratios, lo, m, row_offsets=ro,
                                 max_n=self.max_n, workspace=self.ws, out=self.sout)
            if ev: ev[2].record(st)
            pwlq.quantize_unsigned(x, self.bits, lo, m, self.sout["p"], layout=self.layout,
                                   row_offsets=ro, out=(self.codes, self.mask, None))
            if ev: ev[3].record(st)
            pwlq.dequantize_unsigned(self.codes, self.mask, self.bits, lo, m, self.sout["p"],
                                     C=w.C, n=self.dense_n, layout=self.layout, row_offsets=ro,
                                     out=self.y)
            if ev: ev[4].record(st)
            return
        pwlq.absmax(x, row_offsets=ro, out=m)
        if ev: ev[1].record(st)
        pwlq.search(x, self.bits, self.ratios, m=m, row_offsets=ro, max_n=self.max_n,
                    workspace=self.ws, out=self.sout)
        if ev: ev[2].record(st)
        pwlq.quantize(x, self.bits, m, self.sout["p"], layout=self.layout, row_offsets=ro,
                      out=(self.codes, self.mask, None))
        if ev: ev[3].record(st)
        pwlq.dequantize(self.codes, self.mask, self.bits, m, self.sout["p"], C=w.C, n=self.dense_n,
                        layout=self.layout, row_offsets=ro, out=self.y)
        if ev: ev[4].record(st)

    def timed_steps(self, steps, flush, warmup=0, barrier=None):
        """Stage times [steps, 4] in ms; the L2 is evicted before every step."""
        torch = self.torch
        for _ in range(warmup):
            flush.fill_(1)
            self.step()
        if barrier: barrier()
        events = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(steps)]
        for i in range(steps):
            flush.fill_(i & 0xFF)                 # evict the 126 MB L2 between timed steps
            self.step(events[i])
        if barrier: barrier()
        else: torch.cuda.synchronize()
        return np.array([[ev[j].elapsed_time(ev[j + 1]) for j in range(4)] for ev in events])

    def streaming(self, reps=10, multi=False):
        """The three HBM-bound kernels back to back on the workload's rows repeated until they
        exceed L2 three times over (no eviction pass needed, no cold first wave per launch).
        multi: also the three-breakpoint quantize / dequantize (signed scheme) on the same rows,
        with breakpoints at 0.2 / 0.45 / 0.75 of every row's range."""
        torch, pwlq, w = self.torch, self.pwlq, self.w
        copies = max(1, -(-(3 * L2_BYTES) // (w.total * 4)))
        ro_b = None                                  # equally long rows stay a dense matrix
        if self.dense_n is None:
            offs = [w.row_offsets[:-1] + k * w.total for k in range(copies)]
            ro_b = torch.from_numpy(np.concatenate(offs + [np.array([copies * w.total])])).to(self.dev)
        x_b = self.x.reshape(-1).repeat(copies)
        if self.dense_n is not None:
            x_b = x_b.view(copies * w.C, self.dense_n)
        tot_b = x_b.numel()
        m_b = torch.empty(copies * w.C, dtype=torch.float32, device=self.dev)
        codes_b = torch.empty(pwlq.code_bytes(tot_b, self.bits, self.layout), dtype=torch.uint8,
                              device=self.dev)
        mask_b = torch.empty((tot_b + 7) // 8, dtype=torch.uint8, device=self.dev)
        y_b = torch.empty(tot_b, dtype=torch.float32, device=self.dev)
        pwlq.absmax(x_b, row_offsets=ro_b, out=m_b)
        p_b = self.sout["p"].repeat(copies)
        io = tot_b * 4 + codes_b.numel() + mask_b.numel()
        calls = {
            "absmax": (lambda: pwlq.absmax(x_b, row_offsets=ro_b, out=m_b), tot_b * 4),
            "quantize": (lambda: pwlq.quantize(x_b, self.bits, m_b, p_b, layout=self.layout,
                                               row_offsets=ro_b, out=(codes_b, mask_b, None)), io),
            "quantize_fused": (lambda: pwlq.quantize(x_b, self.bits, m_b, p_b, layout=self.layout,
                                                     row_offsets=ro_b,
                                                     out=(codes_b, mask_b, y_b)), io + tot_b * 4),
            "dequantize": (lambda: pwlq.dequantize(codes_b, mask_b, self.bits, m_b, p_b,
                                                   C=copies * w.C, n=self.dense_n,
                                                   layout=self.layout, row_offsets=ro_b, out=y_b),
                           io),
        }
        out = {"rows": f"the workload's rows x{copies} ({tot_b * 4 >> 20} MiB, larger than L2), "
                       "back to back, no eviction"}
        st = torch.cuda.current_stream()

        def timed(fn, n):
            for _ in range(3):
                fn()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            a.record(st)
            for _ in range(n):
                fn()
            b.record(st)
            torch.cuda.synchronize()
            return a.elapsed_time(b) / n

        for name, (fn, nbytes) in calls.items():
            out[name] = {"gbs": nbytes / (timed(fn, reps) * 1e-3) / 1e9}
        if multi and not self.unsigned:
            p3_b = torch.stack([m_b * 0.2, m_b * 0.45, m_b * 0.75], dim=1).contiguous()
            reg_b = torch.empty((tot_b + 3) // 4, dtype=torch.uint8, device=self.dev)
            io3 = tot_b * 4 + codes_b.numel() + reg_b.numel()
            tcalls = {
                "quantize3": lambda: pwlq.quantize3(x_b, self.bits, m_b, p3_b, layout=self.layout,
                                                    row_offsets=ro_b, out=(codes_b, reg_b, None)),
                "dequantize3": lambda: pwlq.dequantize3(codes_b, reg_b, self.bits, m_b, p3_b,
                                                        C=copies * w.C, n=self.dense_n,
                                                        layout=self.layout, row_offsets=ro_b, out=y_b),
            }
            out["three_breakpoints"] = {
                name: {"gbs": io3 / (timed(fn, reps) * 1e-3) / 1e9} for name, fn in tcalls.items()}
            del p3_b, reg_b
        if self.dense_n is None or self.dense_n < 4096:
            # several rows per span of 4096 values: the same calls with the layout's row maps
            # built once (pwlq_rowmap_build) instead of inside every kernel
            Cb, nb = copies * w.C, (self.dense_n or 0)
            rmap = pwlq.rowmap_build(Cb, tot_b, row_offsets=ro_b, n=nb, device=self.dev)
            build_ms = timed(lambda: pwlq.rowmap_build(Cb, tot_b, row_offsets=ro_b, n=nb, out=rmap), 3)
            mcalls = {
                "absmax": (lambda: pwlq.absmax(x_b, row_offsets=ro_b, out=m_b, rowmap=rmap), tot_b * 4),
                "quantize": (lambda: pwlq.quantize(x_b, self.bits, m_b, p_b, layout=self.layout,
                                                   row_offsets=ro_b, out=(codes_b, mask_b, None),
                                                   rowmap=rmap), io),
                "quantize_fused": (lambda: pwlq.quantize(x_b, self.bits, m_b, p_b, layout=self.layout,
                                                         row_offsets=ro_b, out=(codes_b, mask_b, y_b),
                                                         rowmap=rmap), io + tot_b * 4),
                "dequantize": (lambda: pwlq.dequantize(codes_b, mask_b, self.bits, m_b, p_b, C=Cb,
                                                       n=self.dense_n, layout=self.layout,
                                                       row_offsets=ro_b, out=y_b, rowmap=rmap), io),
            }
            mapped = {"row_maps": f"built once per layout by pwlq_rowmap_build "
                                  f"({rmap.numel() >> 10} KiB, {build_ms * 1e3:.1f} us), not timed"}
            for name, (fn, nbytes) in mcalls.items():
                mapped[name] = {"gbs": nbytes / (timed(fn, reps) * 1e-3) / 1e9}
            out["mapped"] = mapped
        return out

    def kernels_per_step(self):
        """Kernels of this library per step: abs-max (a second launch turns the keys of min/max
        into values), the search launches (a dense matrix: the one for its row length; ragged rows:
        one per row-length class that begins at or below the longest row -- the library does not
        look at the lengths), the two combine launches when a row exceeds one tile, quantize,
        dequantize."""
        w, max_n = self.w, self.max_n
        tiled = max_n > 8192 or (max_n > 1024 and w.C * -(-max_n // 8192) < 296)
        if self.K > 1024 or self.dense_n is not None:
            classes = 1
        elif tiled and max_n <= 8192:
            classes = 2                                 # one launch for all rows above 64 values
        else:
            classes = sum(max_n >= lo for lo in (0, 65, 513, 2305))
        return 1 + int(self.unsigned) + classes + (2 if tiled else 0) + 2


STREAM_KEYS = ("absmax", "quantize", "quantize_fused", "dequantize")


def add_fracs(s, hbm):
    """Fractions of the copy peak beside the GB/s of a streaming() result (both call forms)."""
    for d in (s, s.get("mapped", {})):
        for k in STREAM_KEYS:
            if k in d:
                d[k]["frac"] = d[k]["gbs"] / hbm
    for v in s.get("three_breakpoints", {}).values():
        v["frac"] = v["gbs"] / hbm
    return s


def stream_fracs(s, hbm):
    out = {k: s[k]["gbs"] / hbm for k in STREAM_KEYS}
    if "mapped" in s:
        out["mapped"] = {k: s["mapped"][k]["gbs"] / hbm for k in STREAM_KEYS}
    return out


def timed_call(torch, fn, flush, reps=5):
    """Median ms of single cold launches (L2 evicted before each)."""
    ts = []
    st = torch.cuda.current_stream()
    for _ in range(reps + 2):
        flush.fill_(1)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(st); fn(); b.record(st)
        torch.cuda.synchronize()
        ts.append(a.elapsed_time(b))
    return float(np.median(ts[2:]))


def extras(torch, pwlq, path: DevicePath, flush, hbm, K2=32):
    """The calls beyond the four-call path, on the headline workload's rows (single cold launches):
    two-breakpoint pair search with its quantize / dequantize, analytic selection, bias correction
    with the corrected dequantize, dense (b+1)-bit stream; and the streaming kernels on dense rows
    of 147 values (row starts off every vector boundary)."""
    w, x, ro, m, bits = path.w, path.x, path.ro, path.m, path.bits
    kw = dict(row_offsets=ro)
    r2 = torch.from_numpy(W.ratio_grid(K2)).to(path.dev)
    out = {}
    ws2 = None
    try:
        s2 = pwlq.search2(x, bits, r2, m, max_n=path.max_n, **kw)
        ws2 = s2["workspace"]
        pairs = K2 * (K2 - 1) // 2
        t = timed_call(torch, lambda: pwlq.search2(x, bits, r2, m, max_n=path.max_n, workspace=ws2,
                                                   **kw), flush)
        one = pwlq.search(x, bits, r2, m=m, max_n=path.max_n, **kw)
        gain = float((one["err"].double().sum() / s2["err"].double().sum()).item())
        out["search2"] = {"K": K2, "pairs": pairs, "ms": t,
                          "t_value_pairs_per_s": w.total * pairs / (t * 1e-3) / 1e12,
                          "sse_one_over_two_breakpoints": gain}
        codes, region, _ = pwlq.quantize2(x, bits, m, s2["p1"], s2["p2"], layout=1, **kw)
        nb = w.total * 4 + codes.numel() + region.numel()
        t = timed_call(torch, lambda: pwlq.quantize2(x, bits, m, s2["p1"], s2["p2"], layout=1,
                                                     out=(codes, region, None), **kw), flush)
        out["quantize2"] = {"ms": t, "hbm_cold_frac": nb / (t * 1e-3) / 1e9 / hbm}
        y = path.y
        t = timed_call(torch, lambda: pwlq.dequantize2(codes, region, bits, m, s2["p1"], s2["p2"],
                                                       C=w.C, n=path.dense_n, layout=1, out=y, **kw),
                       flush)
        out["dequantize2"] = {"ms": t, "hbm_cold_frac": nb / (t * 1e-3) / 1e9 / hbm}
        # three breakpoints: the pair search's terms plus O(K^2) per row
        s3 = pwlq.search3(x, bits, r2, m, max_n=path.max_n, workspace=ws2, **kw)
        t = timed_call(torch, lambda: pwlq.search3(x, bits, r2, m, max_n=path.max_n, workspace=ws2,
                                                   **kw), flush)
        triples = K2 * (K2 - 1) * (K2 - 2) // 6
        out["search3"] = {"K": K2, "triples": triples, "ms": t,
                          "sse_two_over_three_breakpoints":
                              float((s2["err"].double().sum() / s3["err"].double().sum()).item())}
        c3, g3, _ = pwlq.quantize3(x, bits, m, s3["p"], layout=1, **kw)
        t = timed_call(torch, lambda: pwlq.quantize3(x, bits, m, s3["p"], layout=1,
                                                     out=(c3, g3, None), **kw), flush)
        out["quantize3"] = {"ms": t, "hbm_cold_frac": nb / (t * 1e-3) / 1e9 / hbm}
        t = timed_call(torch, lambda: pwlq.dequantize3(c3, g3, bits, m, s3["p"], C=w.C,
                                                       n=path.dense_n, layout=1, out=y, **kw), flush)
        out["dequantize3"] = {"ms": t, "hbm_cold_frac": nb / (t * 1e-3) / 1e9 / hbm}
        del c3, g3
        # the pair search on one long row (a tensor quantized per layer): tiles of 8192 values
        wl = W.relu_activation()
        xl = torch.from_numpy(wl.x).to(path.dev).view(1, -1)
        ml = pwlq.absmax(xl)
        sl = pwlq.search2(xl, bits, r2, ml)
        t = timed_call(torch, lambda: pwlq.search2(xl, bits, r2, ml, workspace=sl["workspace"]),
                       flush, reps=3)
        out["search2_one_row_of_25.7M"] = {"K": K2, "pairs": pairs, "ms": t,
                                           "t_value_pairs_per_s": wl.total * pairs / (t * 1e-3) / 1e12}
        del xl, sl, wl
    except pwlq.PwlqError as e:
        out["search2"] = {"skipped": str(e)}
    p = path.sout["p"]
    t = timed_call(torch, lambda: pwlq.select_analytic(x, m, pwlq.MODEL_GAUSS_ROOT,
                                                       max_n=path.max_n, **kw), flush)
    out["select_analytic"] = {"ms": t, "hbm_cold_frac": w.total * 4 / (t * 1e-3) / 1e9 / hbm}
    t = timed_call(torch, lambda: pwlq.bias_correction(x, bits, m, p, max_n=path.max_n, **kw), flush)
    out["bias_correction"] = {"ms": t, "hbm_cold_frac": w.total * 4 / (t * 1e-3) / 1e9 / hbm}
    xi, beta = pwlq.bias_correction(x, bits, m, p, max_n=path.max_n, **kw)
    c8, k8, _ = pwlq.quantize(x, bits, m, p, layout=0, **kw)
    b8 = w.total * 4 + c8.numel() + k8.numel()
    t = timed_call(torch, lambda: pwlq.dequantize_bc(c8, k8, bits, m, p, xi, beta, C=w.C,
                                                     n=path.dense_n, out=path.y, **kw), flush)
    out["dequantize_bc"] = {"ms": t, "hbm_cold_frac": b8 / (t * 1e-3) / 1e9 / hbm}
    dense = pwlq.pack_dense(c8, k8, bits)
    bp = c8.numel() + k8.numel() + dense.numel()
    t = timed_call(torch, lambda: pwlq.pack_dense(c8, k8, bits, out=dense), flush)
    out["pack_dense"] = {"ms": t, "hbm_cold_frac": bp / (t * 1e-3) / 1e9 / hbm}
    t = timed_call(torch, lambda: pwlq.unpack_dense(dense, w.total, bits), flush)
    out["unpack_dense"] = {"ms": t, "hbm_cold_frac": bp / (t * 1e-3) / 1e9 / hbm}
    del c8, k8, dense
    # streaming kernels on dense rows of 147 values, 512 MB
    n147 = (1 << 27) // 147
    rng = np.random.default_rng(147)
    w147 = W.Workload("dense_rows_of_147", (rng.standard_normal(n147 * 147) * 0.02).astype(np.float32),
                      np.arange(n147 + 1, dtype=np.int64) * 147, 4, 16)
    p147 = DevicePath(torch, pwlq, w147, path.dev)
    pwlq.absmax(p147.x, out=p147.m)
    p147.sout["p"].copy_(p147.m * 0.3)
    s = p147.streaming(reps=5)
    out["hbm_streaming_frac_rows_of_147"] = stream_fracs(s, hbm)
    return out


def summarize(path: DevicePath, stage_ms, hbm, peak_measured, issued=None):
    """Per-workload figures from stage times [steps, 4]."""
    mean = stage_ms.mean(axis=0)
    ec = path.elem_cand
    search_s = mean[1] * 1e-3
    achieved = LANE_OPS_PER_ELEM_CAND * ec / search_s / 1e12
    io = path.io_bytes()
    out = {"bits": path.bits, "K": path.K, "rows": path.w.C, "values": path.w.total,
           "ms_per_step": float(mean.sum()),
           "stages_ms": {"absmax": float(mean[0]), "search": float(mean[1]),
                         "quantize": float(mean[2]), "dequantize": float(mean[3])},
           "gelem_cand_per_s": ec / (mean.sum() * 1e-3) / 1e9,
           "search_gelem_cand_per_s": ec / search_s / 1e9,
           "search_frac": achieved / ALU_PEAK_TLANEOPS,
           "search_frac_of_measured_peak": achieved / peak_measured if peak_measured else None,
           "hbm_cold_frac": {"absmax": path.w.total * 4 / (mean[0] * 1e-3) / 1e9 / hbm,
                             "quantize": io / (mean[2] * 1e-3) / 1e9 / hbm,
                             "dequantize": io / (mean[3] * 1e-3) / 1e9 / hbm}}
    if issued is not None:
        out["search_frac_issued"] = issued * ec / search_s / 1e12 / ALU_PEAK_TLANEOPS
    return out


def run_ours(args, rank, world, local_rank):
    import torch
    from paper_2002_00104_b200 import pwlq
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    pwlq.load_library()
    dev = torch.device("cuda", local_rank)
    stream = torch.cuda.current_stream()
    peaks, peak_kind = measured_peaks()
    hbm = float(peaks["hbm_gbs"])
    gpu_index = (local_rank if "CUDA_VISIBLE_DEVICES" not in os.environ else
                 int(os.environ["CUDA_VISIBLE_DEVICES"].split(",")[local_rank]))

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    w = make_workload(args, None if world == 1 else 1000 + 17 * rank)
    path = DevicePath(torch, pwlq, w, dev, args.scheme)
    if args.leg == "streaming":
        # only the HBM-bound kernels back to back (a small case for a profiler: few launches)
        pwlq.absmax(path.x, row_offsets=path.ro, out=path.m)
        path.sout["p"].copy_(path.m * 0.3)
        s = path.streaming(reps=args.reps, multi=True)
        s["workload"] = w.name
        add_fracs(s, hbm)
        s["device_status"] = pwlq.device_status()
        print(json.dumps({"leg": "streaming", "hbm_streaming": s}), flush=True)
        return
    unsigned = path.unsigned
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    warmup = max(3, args.warmup)

    # ---- the timed region: K steps, L2 evicted before each, clocks sampled meanwhile
    for _ in range(warmup):
        flush.fill_(1)
        path.step()
    barrier()
    sampler = ClockSampler(gpu_index).start()
    stage_ms = path.timed_steps(args.steps, flush, barrier=barrier)
    clocks = sampler.stop()
    total_ms = float(stage_ms.sum())
    status = pwlq.search_status(path.ws) | pwlq.device_status()

    # ---- end to end through the host-buffer entry point (copies inside the timed region)
    max_n, dense_n, layout = path.max_n, path.dense_n, path.layout
    scratch = torch.empty(pwlq.encode_host_scratch_bytes(w.C, w.total, max_n, w.K),
                          dtype=torch.uint8, device=dev)
    hx = torch.from_numpy(w.x).pin_memory()
    hro = None if dense_n is not None else torch.from_numpy(w.row_offsets).pin_memory()
    hr = torch.from_numpy(path.ratios_np).pin_memory()
    hout = {"m": torch.empty(w.C, dtype=torch.float32).pin_memory(),
            "lo": torch.empty(w.C if unsigned else 0, dtype=torch.float32).pin_memory(),
            "p": torch.empty(w.C, dtype=torch.float32).pin_memory(),
            "err": torch.empty(w.C, dtype=torch.float32).pin_memory(),
            "idx": torch.empty(w.C, dtype=torch.int32).pin_memory(),
            "codes": torch.empty(path.codes.numel(), dtype=torch.uint8).pin_memory(),
            "mask": torch.empty(path.mask.numel(), dtype=torch.uint8).pin_memory()}
    h2d = hx.numel() * 4 + (0 if hro is None else hro.numel() * 8) + hr.numel() * 4
    d2h = sum(t.numel() * t.element_size() for t in hout.values())
    hout["hi"] = hout["m"]

    def encode():
        if unsigned:
            pwlq.encode_host_unsigned(hx, hro, w.C, max_n, w.bits, hr, hout, layout, scratch)
        else:
            pwlq.encode_host(hx, hro, w.C, max_n, w.bits, hr, hout, layout, scratch)

    e2e_steps = max(3, min(args.steps, 10))
    for _ in range(2):
        encode()
    barrier()
    e2e_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
              for _ in range(e2e_steps)]
    for a, b in e2e_ev:
        flush.fill_(3)
        a.record(stream)
        encode()
        b.record(stream)
    barrier()
    e2e_ms = float(sum(a.elapsed_time(b) for a, b in e2e_ev))
    # the end-to-end outputs must equal the resident-path outputs (same kernels, same inputs)
    same = bool(torch.equal(hout["codes"], path.codes.cpu()) and
                torch.equal(hout["idx"], path.sout["idx"].cpu()))
    del scratch

    # ---- rank 0, one GPU: the side measurements
    streaming = sustained = others = extra = cold_mapped = None
    peak_measured = peak_detail = None
    if rank == 0 and world == 1 and not args.quick:
        fp = FP32Peak()
        peak_detail = {"fma.rn.f32x2": fp.run(torch, 1), "add.rn.f32x2": fp.run(torch, 2),
                       "fma.rn.f32": fp.run(torch, 0)}
        peak_measured = peak_detail["fma.rn.f32x2"]
        if not unsigned:
            streaming = path.streaming(multi=True)
            if path.dense_n is None or path.dense_n < 4096:
                # the step's three streaming calls as single cold launches, given row maps built
                # once for the layout (the step itself uses the plain calls)
                rmap = pwlq.rowmap_build(w.C, w.total, row_offsets=path.ro, n=path.dense_n or 0,
                                         device=dev)
                p_ = path.sout["p"]
                io_ = path.io_bytes()
                cm = {
                    "absmax": (lambda: pwlq.absmax(path.x, row_offsets=path.ro, out=path.m,
                                                   rowmap=rmap), w.total * 4),
                    "quantize": (lambda: pwlq.quantize(path.x, path.bits, path.m, p_,
                                                       layout=path.layout, row_offsets=path.ro,
                                                       out=(path.codes, path.mask, None),
                                                       rowmap=rmap), io_),
                    "dequantize": (lambda: pwlq.dequantize(path.codes, path.mask, path.bits, path.m,
                                                           p_, C=w.C, n=path.dense_n,
                                                           layout=path.layout, row_offsets=path.ro,
                                                           out=path.y, rowmap=rmap), io_),
                }
                cold_mapped = {}
                for name, (fn, nbytes) in cm.items():
                    t = timed_call(torch, fn, flush)
                    cold_mapped[name] = {"ms": t, "gbs": nbytes / (t * 1e-3) / 1e9,
                                         "frac": nbytes / (t * 1e-3) / 1e9 / hbm}
                del rmap
        # at least two seconds of back-to-back steps: does the figure hold at the sustained clock?
        n_sus = int(np.ceil(2200.0 / max(total_ms / args.steps, 0.05)))
        sampler = ClockSampler(gpu_index).start()
        sus_ms = path.timed_steps(n_sus, flush)
        sus_clocks = sampler.stop()
        mhz = sus_clocks["sm_mhz"] or 1e3 * SM_MAX_GHZ
        sus_search = w.elem_cand / (sus_ms[:, 1].mean() * 1e-3)
        sustained = {"steps": n_sus, "seconds": float(sus_ms.sum() * 1e-3),
                     "ms_per_step": float(sus_ms.sum(axis=1).mean()),
                     "value": w.elem_cand / (sus_ms.sum(axis=1).mean() * 1e-3) / 1e9, "unit": UNIT,
                     "search_gelem_cand_per_s": sus_search / 1e9, "clocks": sus_clocks,
                     "search_frac_at_sampled_clock":
                         LANE_OPS_PER_ELEM_CAND * sus_search /
                         (SM_COUNT * FP32_LANES_PER_SM * mhz * 1e6)}
        if not unsigned:
            extra = extras(torch, pwlq, path, flush, hbm)
        # the other benchmark configurations
        if args.workload == "resnet50" and not (args.bits or args.K) and not unsigned:
            others = {}
            del path.y
            for name in ("single_conv", "mobilenetv2", "relu_activation", "laplace4096"):
                wo = make_workload(args, None, name)
                po = DevicePath(torch, pwlq, wo, dev)
                grids = [(wo.bits, wo.K)] if name != "laplace4096" else \
                    [(b, K) for b in (3, 4, 6, 8) for K in (64, 256, 1024)]
                runs = []
                for bits, K in grids:
                    po.set_grid(bits, K)
                    sm = po.timed_steps(5, flush, warmup=3)
                    r = summarize(po, sm, hbm, peak_measured)
                    r["kernels_per_step"] = po.kernels_per_step()
                    runs.append(r)
                entry = runs[0] if len(runs) == 1 else {"grid": runs}
                po.set_grid(wo.bits, wo.K)
                po.step()
                s = po.streaming(reps=5)
                entry["hbm_streaming_frac"] = stream_fracs(s, hbm)
                entry["device_status"] = pwlq.search_status(po.ws) | pwlq.device_status()
                others[wo.name] = entry
                del po, wo
                torch.cuda.empty_cache()

    # ---- max over ranks
    if dist is not None:
        t = torch.tensor([total_ms, e2e_ms] + stage_ms.sum(axis=0).tolist(), device=dev,
                         dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms, e2e_ms = float(t[0]), float(t[1])
        stage_tot = t[2:].tolist()
    else:
        stage_tot = stage_ms.sum(axis=0).tolist()

    per_step = path.kernels_per_step()
    if rank == 0:
        ec = w.elem_cand
        value = world * ec * args.steps / (total_ms * 1e-3) / 1e9
        search_ms = stage_tot[1] / args.steps
        achieved = LANE_OPS_PER_ELEM_CAND * ec / (search_ms * 1e-3) / 1e12
        issued, center_share, _ = issued_lane_ops(w)
        io = path.io_bytes()

        def gbs(nbytes, ms_total):
            return nbytes / (ms_total / args.steps * 1e-3) / 1e9

        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": warmup, "ms_per_step": total_ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic",
            "config": config_of(w, args.scheme, world),
            "stages_ms": {"absmax": stage_tot[0] / args.steps, "search": search_ms,
                          "quantize": stage_tot[2] / args.steps,
                          "dequantize": stage_tot[3] / args.steps},
            "roofline": {"bound": "alu", "achieved": achieved, "peak": ALU_PEAK_TLANEOPS,
                         "unit": "Tlaneop/s", "frac": achieved / ALU_PEAK_TLANEOPS,
                         "traffic": None,
                         "kernel": "search_sorted_kernel",
                         "peak_source": "148 SMs x 128 FP32 lanes x 1.965 GHz (derived)",
                         "frac_means": "6 lane-ops per evaluation (the definition's count) over peak",
                         "peak_measured": peak_measured, "peak_measured_detail": peak_detail,
                         "frac_of_measured_peak": achieved / peak_measured if peak_measured else None,
                         "lane_ops_issued_per_eval": issued, "center_share": center_share,
                         "frac_issued": issued * ec / (search_ms * 1e-3) / 1e12 / ALU_PEAK_TLANEOPS,
                         "search_gelem_cand_per_s": ec / (search_ms * 1e-3) / 1e9,
                         # the same with the abs-max launch counted into the search's time
                         "frac_with_absmax": LANE_OPS_PER_ELEM_CAND * ec /
                             ((search_ms + stage_tot[0] / args.steps) * 1e-3) / 1e12 /
                             ALU_PEAK_TLANEOPS},
            "hbm_stages": {
                "peak_gbs": hbm, "peak_source": peak_kind,
                "absmax": {"gbs": gbs(w.total * 4, stage_tot[0])},
                "quantize": {"gbs": gbs(io, stage_tot[2])},
                "dequantize": {"gbs": gbs(io, stage_tot[3])}},
            "e2e": {"value": world * ec * e2e_steps / (e2e_ms * 1e-3) / 1e9, "unit": UNIT,
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "ms_per_step": e2e_ms / e2e_steps, "matches_resident_path": same},
            "gpu_launches": per_step * args.steps,
            "kernels_per_step": per_step,
            "clocks": clocks, "device_status": status,
        }
        for k in ("absmax", "quantize", "dequantize"):
            line["hbm_stages"][k]["frac"] = line["hbm_stages"][k]["gbs"] / hbm
        line["hbm_stages"]["timing"] = "one launch per step after the L2 eviction (cold)"
        if world == 1 and not args.quick and cold_mapped is not None:
            line["hbm_stages"]["mapped"] = cold_mapped
        if streaming is not None:
            add_fracs(streaming, hbm)
            streaming["peak_gbs"], streaming["peak_source"] = hbm, peak_kind
            line["hbm_streaming"] = streaming
        if sustained is not None:
            line["sustained"] = sustained
        if others is not None:
            line["workloads"] = others
        if extra is not None:
            line["extras"] = extra
        line["e2e"]["entry_point"] = "pwlq_encode_host_unsigned" if unsigned else "pwlq_encode_host"
        if world == 1 and not args.no_cpu_baseline and not unsigned:
            line["cpu_baseline"] = cpu_baseline_of(w)
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="resnet50", choices=sorted(WORKLOADS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--leg", default="all", choices=["all", "streaming"],
                    help="streaming: only the three HBM-bound kernels back to back on the "
                         "workload's rows repeated beyond L2 (--reps launches each after 3 warm-ups)")
    ap.add_argument("--reps", type=int, default=10)
    ap.add_argument("--quick", action="store_true",
                    help="only the timed steps and the end-to-end leg (no micro-benchmark, "
                         "streaming, sustained or other-workload legs)")
    ap.add_argument("--scheme", default="signed", choices=["signed", "unsigned"],
                    help="unsigned: min/max + one-sided search / quantize / dequantize (b-bit "
                         "levels, no sign bit); a side measurement, not the headline")
    ap.add_argument("--bits", type=int, default=0, help="override the workload's bit-width")
    ap.add_argument("--K", type=int, default=0, help="override the number of candidates")
    ap.add_argument("--rows", type=int, default=0, help="laplace4096 only: number of rows")
    ap.add_argument("--cols", type=int, default=0, help="laplace4096 only: row length")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank, world)
    else:
        run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
