"""Helpers shared by the GPU parity tests."""
import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import torch

SSE_RTOL = 1e-5          # per-candidate squared-error sums: relative tolerance of the parity bar


def dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda()


def sse_atol(n, m):
    """Absolute floor for sums that are (nearly) zero: n values, each off by at most one ulp of m."""
    return float(n) * (2.0 ** -23 * float(m)) ** 2


def check_search(gpu, ora, ratios, m, row_len, want_sse=True):
    """gpu: dict of numpy arrays (p, err, idx, sse); ora: oracle.search result (same rows)."""
    C = ora["idx"].size
    sse_o = ora["sse64"]
    row_len = np.broadcast_to(np.asarray(row_len), (C,))
    atol = np.array([sse_atol(row_len[c], m[c]) for c in range(C)])
    if want_sse:
        diff = np.abs(gpu["sse"].astype(np.float64) - sse_o)
        # + binary32 storage rounding of the delivered sum (half the smallest subnormal at least)
        bound = SSE_RTOL * sse_o + atol[:, None] + 2.0 ** -23 * sse_o + 2.0 ** -150
        bad = diff > bound
        assert not bad.any(), (f"{bad.sum()} SSE entries off; worst rel "
                               f"{(diff / np.maximum(sse_o, 1e-300)).max():.3e}")
    rows = np.arange(C)
    gi, oi = gpu["idx"].astype(np.int64), ora["idx"].astype(np.int64)
    differ = gi != oi
    # a different index is accepted only for a near-tie of the oracle's own sums
    gap = np.abs(sse_o[rows, gi] - sse_o[rows, oi])
    assert np.all(gap[differ] <= SSE_RTOL * sse_o[rows, oi][differ] + atol[differ]), \
        f"{int(differ.sum())} rows differ, worst gap {gap[differ].max() if differ.any() else 0}"
    want_p = (m.astype(np.float32) * ratios[gi]).astype(np.float32)
    want_p[m == 0] = 0.0
    assert np.array_equal(gpu["p"], want_p)
    d = np.abs(gpu["err"].astype(np.float64) - sse_o[rows, gi])
    assert np.all(d <= SSE_RTOL * sse_o[rows, gi] + atol + 2.0 ** -23 * sse_o[rows, gi])
    return int(differ.sum())


def oracle_sse_over_candidates(oracle, x, bits, ratios, m, threads=None):
    """Binary64 sums of ONE long row for every candidate, the single-threaded oracle run on
    slices of the candidate grid by host threads (the C call releases the interpreter lock)."""
    threads = threads or max(1, min(os.cpu_count() or 1, 32))
    chunks = [c for c in np.array_split(np.arange(ratios.size), 4 * threads) if c.size]

    def one(ks):
        return oracle.search(x, bits, np.ascontiguousarray(ratios[ks]), m=m)["sse64"][0]

    with ThreadPoolExecutor(threads) as ex:
        return np.concatenate(list(ex.map(one, chunks)))
