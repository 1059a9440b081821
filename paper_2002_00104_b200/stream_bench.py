"""Back-to-back timing of the HBM-bound kernels (abs-max, quantize, dequantize) on inputs larger
than the 126 MB L2, so that every launch streams from HBM without an eviction pass in between.

    python -m paper_2002_00104_b200.stream_bench [--values N] [--reps R] [--only LAYOUT]

Prints one line per (layout, kernel): microseconds per launch and algorithmic GB/s (abs-max:
4 B/value read; quantize and dequantize with packed 4-bit codes: 4 + 0.5 + 0.125 B/value), next to
a device-to-device copy of the same number of floats (8 B/value) as the yardstick.
"""
from __future__ import annotations

import argparse

import numpy as np
import torch

from . import pwlq, workloads as W


def timeit(fn, reps):
    for _ in range(3):
        fn()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(reps):
        fn()
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) / reps * 1e-3


def run(name, x, ro, C, n, reps, bits=4):
    total = x.numel()
    m = pwlq.absmax(x, row_offsets=ro)
    p = (m * 0.3).contiguous()
    codes = torch.empty((total + 1) // 2, dtype=torch.uint8, device="cuda")
    mask = torch.empty((total + 7) // 8, dtype=torch.uint8, device="cuda")
    y = torch.empty(total, dtype=torch.float32, device="cuda")
    t = timeit(lambda: pwlq.absmax(x, row_offsets=ro, out=m), reps)
    print(f"{name:24s} absmax     {t * 1e6:8.1f} us {total * 4 / t / 1e9:8.0f} GB/s")
    t = timeit(lambda: pwlq.quantize(x, bits, m, p, layout=1, row_offsets=ro, out=(codes, mask, None)), reps)
    print(f"{name:24s} quantize   {t * 1e6:8.1f} us {total * 4.625 / t / 1e9:8.0f} GB/s")
    t = timeit(lambda: pwlq.dequantize(codes, mask, bits, m, p, C=C, n=n, layout=1, row_offsets=ro, out=y), reps)
    print(f"{name:24s} dequantize {t * 1e6:8.1f} us {total * 4.625 / t / 1e9:8.0f} GB/s")
    z = torch.empty_like(y)
    t = timeit(lambda: z.copy_(y), reps)
    print(f"{name:24s} d2d copy   {t * 1e6:8.1f} us {total * 8 / t / 1e9:8.0f} GB/s")
    assert pwlq.device_status() == 0


def tiled(w, copies):
    offs = [w.row_offsets[:-1] + k * w.total for k in range(copies)] + [np.array([copies * w.total])]
    return torch.from_numpy(np.tile(w.x, copies)).cuda(), torch.from_numpy(np.concatenate(offs)).cuda()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--values", type=int, default=1 << 27, help="values per dense tensor (512 MB)")
    ap.add_argument("--reps", type=int, default=10)
    ap.add_argument("--only", default=None,
                    help="run only the layouts whose name contains this text (e.g. 'resnet50')")
    args = ap.parse_args()
    N = args.values

    def wanted(name):
        return args.only is None or args.only in name

    if any(wanted(name) for name in ("dense, 1 row", "dense, rows of 4096", "dense, rows of 147")):
        g = torch.Generator(device="cuda")
        g.manual_seed(0)
        x = torch.randn(N, device="cuda", generator=g) * 0.02
        if wanted("dense, 1 row"):
            run("dense, 1 row", x.view(1, N), None, 1, N, args.reps)
        if wanted("dense, rows of 4096"):
            run("dense, rows of 4096", x.view(N // 4096, 4096), None, N // 4096, 4096, args.reps)
        if wanted("dense, rows of 147"):
            run("dense, rows of 147", x[:147 * (N // 147)].view(N // 147, 147), None, N // 147, 147,
                args.reps)
        del x
    if wanted("ragged, resnet50 x5"):
        xr, ro = tiled(W.resnet50(), 5)
        run("ragged, resnet50 x5", xr, ro, None, None, args.reps)
    if wanted("ragged, mobilenetv2 x30"):
        xr, ro = tiled(W.mobilenetv2(), 30)
        run("ragged, mobilenetv2 x30", xr, ro, None, None, args.reps, bits=3)


if __name__ == "__main__":
    main()
