"""Timing of the calls beyond the one-breakpoint path on ResNet-50 weight shapes: the two-breakpoint
pair search with its quantize / dequantize, bias correction with the corrected dequantize, and the
dense (b+1)-bit stream.

    python -m paper_2002_00104_b200.extras_bench [--K 32] [--bits 4] [--reps 5]

Prints milliseconds per call and, for the search, value-pair evaluations per second: every value
of a row is quantized once under each of the K (K - 1) / 2 breakpoint pairs.  The kernel reaches
that result with fewer operations (the error of a pair splits into a center, a middle and a tail
term, and the center and tail terms are shared between pairs), so the figure is an algorithmic
rate, not a count of executed instructions.
"""
from __future__ import annotations

import argparse

import numpy as np
import torch

from . import pwlq, workloads as W


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--K", type=int, default=32)
    ap.add_argument("--bits", type=int, default=4)
    ap.add_argument("--reps", type=int, default=5)
    args = ap.parse_args()
    w = W.resnet50()
    x = torch.from_numpy(w.x).cuda()
    ro = torch.from_numpy(w.row_offsets).cuda()
    max_n = int(np.diff(w.row_offsets).max())
    ratios = torch.from_numpy(W.ratio_grid(args.K)).cuda()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    m = pwlq.absmax(x, row_offsets=ro)
    out = pwlq.search2(x, args.bits, ratios, m, row_offsets=ro, max_n=max_n)
    codes, region, _ = pwlq.quantize2(x, args.bits, m, out["p1"], out["p2"], layout=1, row_offsets=ro)
    y = pwlq.dequantize2(codes, region, args.bits, m, out["p1"], out["p2"], layout=1, row_offsets=ro)

    def timed(fn):
        ts = []
        for _ in range(args.reps + 2):
            flush.fill_(1)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(); fn(); b.record()
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b))
        return float(np.median(ts[2:]))

    one = pwlq.search(x, args.bits, ratios, m=m, row_offsets=ro, max_n=max_n)
    t1 = timed(lambda: pwlq.search(x, args.bits, ratios, m=m, row_offsets=ro, max_n=max_n))
    t2 = timed(lambda: pwlq.search2(x, args.bits, ratios, m, row_offsets=ro, max_n=max_n))
    tq = timed(lambda: pwlq.quantize2(x, args.bits, m, out["p1"], out["p2"], layout=1,
                                      row_offsets=ro, out=(codes, region, None)))
    td = timed(lambda: pwlq.dequantize2(codes, region, args.bits, m, out["p1"], out["p2"], layout=1,
                                        row_offsets=ro, out=y))
    pairs = args.K * (args.K - 1) // 2
    gain = float((one["err"].double().sum() / out["err"].double().sum()).item())
    nbytes = w.total * 4 + codes.numel() + region.numel()
    print(f"resnet50 shapes, {w.C} rows, {w.total} values, b = {args.bits}, K = {args.K} ({pairs} pairs)")
    print(f"search  (1 breakpoint)  {t1:8.3f} ms  {w.total * args.K / t1 / 1e9:8.2f} T value-candidates/s")
    print(f"search2 (2 breakpoints) {t2:8.3f} ms  {w.total * pairs / t2 / 1e9:8.2f} T value-pairs/s")
    print(f"quantize2               {tq:8.3f} ms  {nbytes / tq / 1e6:8.0f} GB/s")
    print(f"dequantize2             {td:8.3f} ms  {nbytes / td / 1e6:8.0f} GB/s")
    print(f"summed squared error, one breakpoint / two breakpoints: {gain:.2f}")
    # bias correction on the one-breakpoint result; dense stream of its codes
    ws = torch.empty(max(256, int(pwlq.load_library().pwlq_bias_workspace_bytes(w.C, max_n))),
                     dtype=torch.uint8, device="cuda")
    xi, beta = pwlq.bias_correction(x, args.bits, m, one["p"], row_offsets=ro, max_n=max_n,
                                    workspace=ws)
    c8, k8, _ = pwlq.quantize(x, args.bits, m, one["p"], layout=0, row_offsets=ro)
    dense = pwlq.pack_dense(c8, k8, args.bits)
    tb = timed(lambda: pwlq.bias_correction(x, args.bits, m, one["p"], row_offsets=ro, max_n=max_n,
                                            workspace=ws))
    tdb = timed(lambda: pwlq.dequantize_bc(c8, k8, args.bits, m, one["p"], xi, beta,
                                           row_offsets=ro, out=y))
    tp = timed(lambda: pwlq.pack_dense(c8, k8, args.bits, out=dense))
    tu = timed(lambda: pwlq.unpack_dense(dense, w.total, args.bits))
    b8 = w.total * 4 + c8.numel() + k8.numel()
    bp = c8.numel() + k8.numel() + dense.numel()
    print(f"bias_correction         {tb:8.3f} ms  {w.total * 4 / tb / 1e6:8.0f} GB/s")
    print(f"dequantize_bc           {tdb:8.3f} ms  {b8 / tdb / 1e6:8.0f} GB/s")
    print(f"pack_dense              {tp:8.3f} ms  {bp / tp / 1e6:8.0f} GB/s")
    print(f"unpack_dense            {tu:8.3f} ms  {bp / tu / 1e6:8.0f} GB/s")
    assert pwlq.device_status() == 0


if __name__ == "__main__":
    main()
