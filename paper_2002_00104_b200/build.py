"""Builds ``libpwlq.so`` (the C-ABI CUDA library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libpwlq.so")
PEAK_LIB = os.path.join(HERE, "libpwlq_peak.so")     # FP32 micro-benchmark, loaded by bench.py only
PEAK_SOURCES = ["fp32_peak.cu"]
SOURCES = ["pwlq_api.cu", "pwlq_absmax.cu", "pwlq_search.cu", "pwlq_quantize.cu",
           "pwlq_noalloc.cu", "pwlq_select.cu", "pwlq_search2.cu", "pwlq_bias.cu", "pwlq_rowmap.cu"]
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
    "-fmad=false",            # no implicit FMA contraction: every fused op is an explicit fmaf
    "--shared", "-Xcompiler", "-fPIC", "-cudart", "static",
    "--threads", "0",         # the source files are compiled side by side
]


def _stale(lib: str) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)]
    deps += [os.path.join(HERE, "..", "include", "pwlq.h"), os.path.abspath(__file__)]
    return any(os.path.getmtime(d) > t for d in deps)


def _nvcc(sources, lib: str, verbose: bool) -> None:
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + \
          [os.path.join(CSRC, s) for s in sources] + ["-o", lib]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    if verbose:
        print(res.stderr)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compiles the library (and the benchmark's FP32 micro-benchmark) if a source is newer."""
    if force or _stale(LIB):
        _nvcc(SOURCES, LIB, verbose)
    if force or _stale(PEAK_LIB):
        _nvcc(PEAK_SOURCES, PEAK_LIB, verbose)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
