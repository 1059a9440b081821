#!/usr/bin/env python
"""Benchmark of the PWLQ hot path on B200.

One step = one pass of the whole path over one batch of synthetic tensors:
abs-max -> K-candidate breakpoint search -> quantize (packed codes + region mask) -> dequantize.
The default workload is the full set of ResNet-50 v1.5 conv + fc weight shapes quantized per
output channel at 4 bits with K = 256 candidates (27 560 rows, 25.5 M values, 6.53 G
value-candidate evaluations per step).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

Prints ONE JSON line.  `value` is value-candidate evaluations per second of the whole step with
inputs resident in HBM; `e2e` is the same metric through the host-buffer entry point with the
host<->device copies inside the timed region; `hbm_stages` gives the three HBM-bound kernels as
timed inside the step (one cold launch each after the L2 eviction), `hbm_streaming` the same
kernels back to back on the workload's rows repeated until they exceed L2.  With N > 1 (torchrun) every rank processes its
own batch (rows are independent: no collective on the data path) and the slowest rank's time
counts.  `--impl reference` times the CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
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
# dram__bytes_read.sum + dram__bytes_write.sum of the search kernels of ONE step, from the ncu
# capture summarised in profiles/search_sorted_kernel_resnet50.md (103.31 MB read, 0.33 MB
# written; the values themselves are 102.0 MB).  Keyed by (workload, bits, K); None elsewhere.
SEARCH_DRAM_BYTES = {("resnet50", 4, 256): 103.64e6}

WORKLOADS = {
    "resnet50": W.resnet50,
    "single_conv": W.single_conv,
    "mobilenetv2": W.mobilenetv2,
    "relu_activation": W.relu_activation,
    "laplace4096": W.laplace_matrix,
}


def make_workload(args, seed):
    """The named workload; --bits / --K / --rows / --cols override its defaults (sweeps)."""
    kw = {} if seed is None else {"seed": seed}
    if args.workload == "laplace4096":
        if args.rows: kw["rows"] = args.rows
        if args.cols: kw["cols"] = args.cols
    w = WORKLOADS[args.workload](**kw)
    if args.bits: w.bits = args.bits
    if args.K: w.K = args.K
    return w


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": 6650.0}, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
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
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        self.thread.join(timeout=2)
        sm, mx, reasons = [], [], set()
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                "sw_power_cap"), r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        busy = [s for s in sm if s > 0]
        return {"sm_mhz": statistics.median(busy) if busy else None,
                "sm_max_mhz": max(mx) if mx else None, "reasons": sorted(reasons),
                "samples": len(busy)}


# --------------------------------------------------------------------------- CPU oracle timing
def oracle_sample(w: W.Workload, budget_evals: float):
    """A stratified subset of rows (every s-th row, so each layer shape is represented in
    proportion) holding about `budget_evals` value-candidate evaluations."""
    stride = max(1, int(round(w.elem_cand / budget_evals)))
    if w.C == 1:                       # a single long row: take a prefix of its values
        n = max(1, min(w.total, int(budget_evals // w.K)))
        return [(0, n)], f"first {n} of {w.total} values of the single row, all {w.K} candidates"
    rows = list(range(0, w.C, stride))
    spans = [(int(w.row_offsets[c]), int(w.row_offsets[c + 1])) for c in rows]
    return spans, f"every {stride}th row ({len(rows)} of {w.C} rows), all {w.K} candidates"


def time_oracle(w: W.Workload, spans, threads: int):
    """Times oracle abs-max + search + quantize + dequantize over the sampled rows; rows are
    fanned out over `threads` host threads (the oracle itself is single-threaded C)."""
    import oracle
    oracle.build()
    ratios = W.ratio_grid(w.K)

    def one(span):
        b, e = span
        x = w.x[b:e]
        m = oracle.absmax(x)
        r = oracle.search(x, w.bits, ratios, m=m, want_sse=False)
        codes, mask, _ = oracle.quantize(x, w.bits, m, r["p"], layout=1, want_fake=False)
        oracle.dequantize(codes, mask, w.bits, m, r["p"], C=1, n=e - b, layout=1)
        return (e - b) * w.K

    t0 = time.perf_counter()
    if threads > 1:
        with ThreadPoolExecutor(threads) as ex:
            evals = sum(ex.map(one, spans, chunksize=max(1, len(spans) // (threads * 8))))
    else:
        evals = sum(one(s) for s in spans)
    dt = time.perf_counter() - t0
    return evals, dt


def run_reference(args, rank, world):
    if rank != 0:
        return
    w = make_workload(args, None)
    cores = os.cpu_count() or 1
    # size the per-step sample from a short calibration so that the run ends within minutes
    spans, _ = oracle_sample(w, 2e8)
    ev, dt = time_oracle(w, spans, cores)
    rate = ev / dt
    per_step = min(w.elem_cand, rate * max(2.0, 90.0 / max(1, args.steps + args.warmup)))
    spans, what = oracle_sample(w, per_step)
    for _ in range(args.warmup):
        time_oracle(w, spans, cores)
    tot_ev, tot_dt = 0, 0.0
    for _ in range(args.steps):
        ev, dt = time_oracle(w, spans, cores)
        tot_ev += ev; tot_dt += dt
    val = tot_ev / tot_dt / 1e9
    line = {"metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * tot_dt / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic", "impl": "reference",
            "config": {"workload": w.name, "bits": w.bits, "K": w.K, "rows": w.C,
                       "values": w.total, "sample_per_step": what},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": what},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------ GPU arm
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

    w = make_workload(args, None if world == 1 else 1000 + 17 * rank)
    ratios_np = W.ratio_grid(w.K)
    max_n = int(np.diff(w.row_offsets).max())
    dense_n = w.uniform_n()
    layout = pwlq.CODES_PACKED
    dev = torch.device("cuda", local_rank)
    stream = torch.cuda.current_stream()

    # resident inputs and outputs
    x = torch.from_numpy(w.x).to(dev)
    if dense_n is not None:
        x = x.view(w.C, dense_n)
        ro = None
    else:
        ro = torch.from_numpy(w.row_offsets).to(dev)
    ratios = torch.from_numpy(ratios_np).to(dev)
    m = torch.empty(w.C, dtype=torch.float32, device=dev)
    lo = torch.empty(w.C, dtype=torch.float32, device=dev)      # one-sided scheme: range [lo, m]
    unsigned = args.scheme == "unsigned"
    sout = {"p": torch.empty(w.C, dtype=torch.float32, device=dev),
            "err": torch.empty(w.C, dtype=torch.float32, device=dev),
            "idx": torch.empty(w.C, dtype=torch.int32, device=dev), "sse": None}
    ws = torch.empty(max(256, pwlq.search_workspace_bytes(w.C, max_n, w.K)), dtype=torch.uint8,
                     device=dev)
    codes = torch.empty(pwlq.code_bytes(w.total, w.bits, layout), dtype=torch.uint8, device=dev)
    mask = torch.empty((w.total + 7) // 8, dtype=torch.uint8, device=dev)
    y = torch.empty(w.total, dtype=torch.float32, device=dev)
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)

    def step(ev=None):
        """One pass of the whole path; ev = 5 CUDA events to record between the stages."""
        if ev: ev[0].record(stream)
        if unsigned:
            pwlq.minmax(x, row_offsets=ro, out=(lo, m))
            if ev: ev[1].record(stream)
            pwlq.search_unsigned(x, w.bits, ratios, lo, m, row_offsets=ro, max_n=max_n,
                                 workspace=ws, out=sout)
            if ev: ev[2].record(stream)
            pwlq.quantize_unsigned(x, w.bits, lo, m, sout["p"], layout=layout, row_offsets=ro,
                                   out=(codes, mask, None))
            if ev: ev[3].record(stream)
            pwlq.dequantize_unsigned(codes, mask, w.bits, lo, m, sout["p"], C=w.C, n=dense_n,
                                     layout=layout, row_offsets=ro, out=y)
            if ev: ev[4].record(stream)
            return
        pwlq.absmax(x, row_offsets=ro, out=m)
        if ev: ev[1].record(stream)
        pwlq.search(x, w.bits, ratios, m=m, row_offsets=ro, max_n=max_n, workspace=ws, out=sout)
        if ev: ev[2].record(stream)
        pwlq.quantize(x, w.bits, m, sout["p"], layout=layout, row_offsets=ro,
                      out=(codes, mask, None))
        if ev: ev[3].record(stream)
        pwlq.dequantize(codes, mask, w.bits, m, sout["p"], C=w.C, n=dense_n, layout=layout,
                        row_offsets=ro, out=y)
        if ev: ev[4].record(stream)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(3, args.warmup)):
        flush.fill_(1)
        step()
    barrier()

    sampler = ClockSampler(local_rank if "CUDA_VISIBLE_DEVICES" not in os.environ else
                           int(os.environ["CUDA_VISIBLE_DEVICES"].split(",")[local_rank]))
    sampler.start()
    events = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(args.steps)]
    barrier()
    for i in range(args.steps):
        flush.fill_(i & 0xFF)                 # evict the 126 MB L2 between timed steps
        step(events[i])
    barrier()
    stage_ms = np.array([[ev[j].elapsed_time(ev[j + 1]) for j in range(4)] for ev in events])
    step_ms = stage_ms.sum(axis=1)
    total_ms = float(step_ms.sum())
    status = pwlq.search_status(ws)

    # ---- end to end through the host-buffer entry point (copies inside the timed region)
    scratch = torch.empty(pwlq.encode_host_scratch_bytes(w.C, w.total, max_n, w.K),
                          dtype=torch.uint8, device=dev)
    hx = torch.from_numpy(w.x).pin_memory()
    hro = None if dense_n is not None else torch.from_numpy(w.row_offsets).pin_memory()
    hr = torch.from_numpy(ratios_np).pin_memory()
    hout = {"m": torch.empty(w.C, dtype=torch.float32).pin_memory(),
            "p": torch.empty(w.C, dtype=torch.float32).pin_memory(),
            "err": torch.empty(w.C, dtype=torch.float32).pin_memory(),
            "idx": torch.empty(w.C, dtype=torch.int32).pin_memory(),
            "codes": torch.empty(codes.numel(), dtype=torch.uint8).pin_memory(),
            "mask": torch.empty(mask.numel(), dtype=torch.uint8).pin_memory()}
    h2d = hx.numel() * 4 + (0 if hro is None else hro.numel() * 8) + hr.numel() * 4
    d2h = sum(t.numel() * t.element_size() for t in hout.values())
    e2e_steps = max(3, min(args.steps, 10))
    for _ in range(2):
        pwlq.encode_host(hx, hro, w.C, max_n, w.bits, hr, hout, layout, scratch)
    barrier()
    e2e_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
              for _ in range(e2e_steps)]
    for a, b in e2e_ev:
        flush.fill_(3)
        a.record(stream)
        pwlq.encode_host(hx, hro, w.C, max_n, w.bits, hr, hout, layout, scratch)
        b.record(stream)
    barrier()
    e2e_ms = float(sum(a.elapsed_time(b) for a, b in e2e_ev))

    # ---- the three HBM-bound kernels back to back on the workload's rows repeated until they
    # exceed L2 (no eviction pass needed then, and no cold first wave in every launch)
    stream = None
    if rank == 0 and not unsigned:
        copies = max(1, -(-(3 * 126 << 20) // (w.total * 4)))        # >= 3 x the 126 MB L2
        ro_b = None                                  # equally long rows stay a dense matrix
        if dense_n is None:
            offs = [w.row_offsets[:-1] + k * w.total for k in range(copies)]
            ro_b = torch.from_numpy(np.concatenate(offs + [np.array([copies * w.total])])).to(dev)
        x_b = x.reshape(-1).repeat(copies)
        if dense_n is not None:
            x_b = x_b.view(copies * w.C, dense_n)
        m_b = torch.empty(copies * w.C, dtype=torch.float32, device=dev)
        tot_b = x_b.numel()
        codes_b = torch.empty(pwlq.code_bytes(tot_b, w.bits, layout), dtype=torch.uint8, device=dev)
        mask_b = torch.empty((tot_b + 7) // 8, dtype=torch.uint8, device=dev)
        y_b = torch.empty(tot_b, dtype=torch.float32, device=dev)
        pwlq.absmax(x_b, row_offsets=ro_b, out=m_b)
        p_b = sout["p"].repeat(copies)
        calls = {
            "absmax": (lambda: pwlq.absmax(x_b, row_offsets=ro_b, out=m_b), tot_b * 4),
            "quantize": (lambda: pwlq.quantize(x_b, w.bits, m_b, p_b, layout=layout, row_offsets=ro_b,
                                               out=(codes_b, mask_b, None)),
                         tot_b * 4 + codes_b.numel() + mask_b.numel()),
            "dequantize": (lambda: pwlq.dequantize(codes_b, mask_b, w.bits, m_b, p_b, C=copies * w.C,
                                                   n=dense_n, layout=layout, row_offsets=ro_b,
                                                   out=y_b),
                           tot_b * 4 + codes_b.numel() + mask_b.numel()),
        }
        stream = {"rows": f"the workload's rows x{copies} ({tot_b * 4 >> 20} MiB, larger than L2), "
                          "back to back, no eviction"}
        reps = 10
        for name, (fn, nbytes) in calls.items():
            for _ in range(3):
                fn()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            a.record(stream_ := torch.cuda.current_stream())
            for _ in range(reps):
                fn()
            b.record(stream_)
            torch.cuda.synchronize()
            stream[name] = {"gbs": nbytes / (a.elapsed_time(b) / reps * 1e-3) / 1e9}
        del x_b, y_b, codes_b, mask_b
    clocks = sampler.stop()

    # the end-to-end outputs must equal the resident-path outputs (same kernels, same inputs)
    same = bool(torch.equal(hout["codes"], codes.cpu()) and torch.equal(hout["idx"], sout["idx"].cpu()))
    if unsigned:
        same = None          # the host-buffer entry point runs the signed scheme only

    # ---- max over ranks
    if dist is not None:
        t = torch.tensor([total_ms, e2e_ms] + stage_ms.sum(axis=0).tolist(), device=dev,
                         dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms, e2e_ms = float(t[0]), float(t[1])
        stage_tot = t[2:].tolist()
    else:
        stage_tot = stage_ms.sum(axis=0).tolist()

    # kernels of this library per step: abs-max, the search launches (a dense matrix: the one for
    # its row length; ragged rows: one per row-length class that begins at or below the longest
    # row -- the library does not look at the lengths), the two combine launches when a row exceeds
    # one tile, quantize, dequantize
    tiled = max_n > 8192 or (max_n > 1024 and w.C * -(-max_n // 8192) < 296)   # several tiles per row
    if w.K > 1024 or dense_n is not None:
        classes = 1
    elif tiled and max_n <= 8192:
        classes = 2                                     # one launch for all rows above 64 values
    else:
        classes = sum(max_n >= lo for lo in (0, 65, 513, 2305))
    per_step = 1 + classes + (2 if tiled else 0) + 2
    if rank == 0:
        peaks, peak_kind = measured_peaks()
        ec = w.elem_cand
        value = world * ec * args.steps / (total_ms * 1e-3) / 1e9
        search_ms = stage_tot[1] / args.steps
        achieved = LANE_OPS_PER_ELEM_CAND * ec / (search_ms * 1e-3) / 1e12
        q_bytes = w.total * 4 + codes.numel() + mask.numel()
        dq_bytes = w.total * 4 + codes.numel() + mask.numel()
        hbm = float(peaks["hbm_gbs"])

        def gbs(nbytes, ms_total):
            return nbytes / (ms_total / args.steps * 1e-3) / 1e9

        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": total_ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic",
            "config": {"workload": w.name, "bits": w.bits, "K": w.K, "rows": w.C,
                       "values": w.total, "elem_cand_per_step": ec, "code_layout": "packed",
                       "scheme": args.scheme,
                       "l2": f"flushed between steps by writing {L2_FLUSH_BYTES >> 20} MiB",
                       "parallelism": f"independent batches x{world}"},
            "stages_ms": {"absmax": stage_tot[0] / args.steps, "search": search_ms,
                          "quantize": stage_tot[2] / args.steps,
                          "dequantize": stage_tot[3] / args.steps},
            "roofline": {"bound": "alu", "achieved": achieved, "peak": ALU_PEAK_TLANEOPS,
                         "unit": "Tlaneop/s", "frac": achieved / ALU_PEAK_TLANEOPS,
                         "traffic": SEARCH_DRAM_BYTES.get((args.workload, w.bits, w.K)),
                         "kernel": "search_sorted_kernel",
                         "peak_source": "148 SMs x 128 FP32 lanes x 1.965 GHz (derived)",
                         "search_gelem_cand_per_s": ec / (search_ms * 1e-3) / 1e9},
            "hbm_stages": {
                "peak_gbs": hbm, "peak_source": peak_kind,
                "absmax": {"gbs": gbs(w.total * 4, stage_tot[0])},
                "quantize": {"gbs": gbs(q_bytes, stage_tot[2])},
                "dequantize": {"gbs": gbs(dq_bytes, stage_tot[3])}},
            "e2e": {"value": world * ec * e2e_steps / (e2e_ms * 1e-3) / 1e9, "unit": UNIT,
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "ms_per_step": e2e_ms / e2e_steps, "matches_resident_path": same},
            "gpu_launches": (per_step + int(unsigned)) * (args.steps + max(3, args.warmup)) +
                            per_step * (e2e_steps + 2),
            "kernels_per_step": per_step,
            "clocks": clocks, "device_status": status,
        }
        for k in ("absmax", "quantize", "dequantize"):
            line["hbm_stages"][k]["frac"] = line["hbm_stages"][k]["gbs"] / hbm
        line["hbm_stages"]["timing"] = "one launch per step after the L2 eviction (cold)"
        if stream is not None:
            for k in ("absmax", "quantize", "dequantize"):
                stream[k]["frac"] = stream[k]["gbs"] / hbm
            stream["peak_gbs"], stream["peak_source"] = hbm, peak_kind
            line["hbm_streaming"] = stream
        if unsigned:
            line["e2e"]["scheme"] = "signed (the host-buffer entry point has no one-sided form)"
        if world == 1 and not args.no_cpu_baseline and not unsigned:
            cores = os.cpu_count() or 1
            spans, _ = oracle_sample(w, 2e8)                 # short calibration
            ev, dt = time_oracle(w, spans, cores)
            spans, what = oracle_sample(w, min(w.elem_cand, 15.0 * ev / dt))   # about 15 s ...
            ev, dt, passes = 0, 0.0, 0
            while dt < 10.0 and passes < 8:                  # ... repeated if the box is faster
                e1, d1 = time_oracle(w, spans, cores)
                ev += e1; dt += d1; passes += 1
            what += f", {passes} pass(es)"
            line["cpu_baseline"] = {"value": ev / dt / 1e9, "unit": UNIT, "cores": cores,
                                    "kind": "oracle", "sample": what, "seconds": dt}
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
