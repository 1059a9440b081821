"""Row sharding across ranks: host logic, checked with two gloo ranks on CPU.

Each rank runs the whole path on its block of rows (the CPU oracle stands in for the device
kernels here: the point is the partition and the gather), and the gathered per-row results must
equal the single-process results bit for bit."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2002_00104_b200 import shard, workloads as W


def test_partition_is_contiguous_balanced_and_complete():
    w = W.small_mixed(seed=4)
    for ws in (1, 2, 3, 5, 20):
        parts = shard.partition_rows(w.row_offsets, ws)
        assert parts[0][0] == 0 and parts[-1][1] == w.C
        assert all(a[1] == b[0] for a, b in zip(parts, parts[1:]))
        assert all(r0 <= r1 for r0, r1 in parts)
    w = W.mobilenetv2()
    parts = shard.partition_rows(w.row_offsets, 8)
    sizes = [int(w.row_offsets[b] - w.row_offsets[a]) for a, b in parts]
    assert sum(sizes) == w.total
    assert max(sizes) - min(sizes) <= 2 * 1280          # within two longest rows of each other
    x, ro, (r0, r1) = shard.shard(w.x, w.row_offsets, 3, 8)
    assert ro[0] == 0 and ro[-1] == x.size == sizes[3] and ro.size == r1 - r0 + 1


def _worker(rank, world, port, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import oracle
    w = W.small_mixed(seed=9, bits=4, K=32)
    ratios = W.ratio_grid(w.K)
    x, ro, rng = shard.shard(w.x, w.row_offsets, rank, world)
    if ro.size > 1:
        m = oracle.absmax(x, ro)
        r = oracle.search(x, w.bits, ratios, m=m, row_offsets=ro, want_sse=False)
        local = {"m": m, "p": r["p"], "err": r["err"], "idx": r["idx"]}
    else:
        local = {"m": np.zeros(0, np.float32), "p": np.zeros(0, np.float32),
                 "err": np.zeros(0, np.float32), "idx": np.zeros(0, np.int32)}
    full = shard.gather_rows(local, None, dist, rank, world)
    if rank == 0:
        q.put({k: v.tobytes() for k, v in full.items()})
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_reproduce_the_single_process_result():
    import oracle
    oracle.build()
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = q.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    w = W.small_mixed(seed=9, bits=4, K=32)
    m = oracle.absmax(w.x, w.row_offsets)
    r = oracle.search(w.x, w.bits, W.ratio_grid(w.K), m=m, row_offsets=w.row_offsets, want_sse=False)
    assert got["m"] == m.tobytes() and got["p"] == r["p"].tobytes()
    assert got["err"] == r["err"].tobytes() and got["idx"] == r["idx"].tobytes()


# ------------------------------------------------------------------ one row cut across two ranks
def test_partition_of_elements_is_aligned_and_complete():
    for n, ws in ((36864, 2), (25690112, 8), (17, 4), (5, 8), (1000, 3)):
        parts = shard.partition_elements(n, ws)
        assert parts[0][0] == 0 and parts[-1][1] == n
        assert all(a[1] == b[0] for a, b in zip(parts, parts[1:]))
        assert all(b % 8 == 0 for b, _ in parts)


def _split_worker(rank, world, port, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import oracle
    w = W.single_conv()                       # one row of 36 864 values, K = 100
    ratios = W.ratio_grid(w.K)
    b, e = shard.partition_elements(w.total, world)[rank]
    xs = w.x[b:e]
    # the oracle stands in for pwlq_absmax / pwlq_search_partial on this rank's slice
    m = torch.from_numpy(oracle.absmax(xs))
    shard.allreduce_range(m, dist)
    sums = torch.from_numpy(oracle.search(xs, w.bits, ratios, m=m.numpy())["sse64"])
    stacked = shard.gather_partial_sums(sums, dist, world)
    # stand-in for pwlq_search_finish: parts added in rank order, first minimum
    tot = stacked[0].clone()
    for r in range(1, world):
        tot += stacked[r]
    idx = int(torch.argmin(tot[0]))
    q.put((rank, m.numpy().tobytes(), tot.numpy().tobytes(), idx))
    dist.barrier()
    dist.destroy_process_group()


def test_one_row_cut_across_two_ranks_matches_the_single_process_search():
    import oracle
    oracle.build()
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_split_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    # every rank ends with the same range, the same sums (bit for bit) and the same index
    assert got[0][1:] == got[1][1:]
    w = W.single_conv()
    m = oracle.absmax(w.x)
    ref = oracle.search(w.x, w.bits, W.ratio_grid(w.K), m=m)
    assert got[0][1] == m.tobytes()
    tot = np.frombuffer(got[0][2], np.float64)
    assert np.allclose(tot, ref["sse64"][0], rtol=1e-12, atol=0)     # binary64 sums, other order
    assert got[0][3] == int(ref["idx"][0])
