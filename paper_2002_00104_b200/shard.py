"""Splitting one workload's rows across ranks (host logic only, no arithmetic of the method).

Rows are independent (every output of the path is per row), so a multi-GPU run needs no
collective on the data path: each rank takes a contiguous block of rows holding about the same
number of value-candidate evaluations, runs the whole path on it, and the per-row results
(m, p, err, idx: 16 bytes per row) are gathered afterwards if one rank wants them all.
"""
from __future__ import annotations

import numpy as np


def partition_rows(row_offsets: np.ndarray, world_size: int):
    """Contiguous row ranges [(r0, r1)] * world_size with balanced numbers of values.

    The cost of a row is its length (every row sees the same K candidates), so the cut points are
    the rows at which the running number of values crosses k/world_size of the total."""
    row_offsets = np.asarray(row_offsets, dtype=np.int64)
    C = row_offsets.size - 1
    total = int(row_offsets[-1])
    cuts = [0]
    for k in range(1, world_size):
        target = total * k // world_size
        r = int(np.searchsorted(row_offsets, target, side="left"))
        cuts.append(min(max(r, cuts[-1]), C))
    cuts.append(C)
    return [(cuts[k], cuts[k + 1]) for k in range(world_size)]


def shard(x: np.ndarray, row_offsets: np.ndarray, rank: int, world_size: int):
    """This rank's rows: (values, row_offsets rebased to 0, (first_row, last_row + 1))."""
    r0, r1 = partition_rows(row_offsets, world_size)[rank]
    b, e = int(row_offsets[r0]), int(row_offsets[r1])
    return x[b:e], (row_offsets[r0:r1 + 1] - row_offsets[r0]).astype(np.int64), (r0, r1)


def gather_rows(local: dict, ranges, dist, rank: int, world_size: int):
    """All ranks' per-row arrays concatenated in row order (torch.distributed all_gather_object
    on small host arrays; the device path has no collective)."""
    out = [None] * world_size
    dist.all_gather_object(out, {k: np.asarray(v) for k, v in local.items()})
    return {k: np.concatenate([out[r][k] for r in range(world_size)]) for k in local}


# ---------------------------------------------------------------------------- one row, many ranks
# A tensor quantized per layer is ONE row; it does not shard by rows.  Its elements are cut into
# contiguous slices instead.  The range needs one exchange (maximum of the ranks' abs-max values),
# the search a second one (the ranks' per-candidate sums, K binary64 values per row, added in rank
# order so that every rank gets the same bits), after which every rank takes the same argmin.
# Quantize and dequantize are element-wise and need nothing.  The functions below are the two
# exchanges; the arithmetic between them is the library's (pwlq_absmax, pwlq_search_partial,
# pwlq_search_finish).

def partition_elements(n: int, world_size: int, align: int = 8):
    """Contiguous element ranges [(b, e)] * world_size of a row of n values, cut at multiples of
    `align` (so that every slice keeps the vector and byte alignment of codes and region bits)."""
    cuts = [0]
    for k in range(1, world_size):
        c = (n * k // world_size) // align * align
        cuts.append(min(max(c, cuts[-1]), n))
    cuts.append(n)
    return [(cuts[k], cuts[k + 1]) for k in range(world_size)]


def allreduce_range(m_local, dist, group=None):
    """Range of the whole rows from the ranks' ranges of their slices: element-wise maximum
    (exact and order-free).  m_local: float32 tensor [C] on the backend's device; in place."""
    dist.all_reduce(m_local, op=dist.ReduceOp.MAX, group=group)
    return m_local


def gather_partial_sums(sums_local, dist, world_size: int, group=None):
    """All ranks' per-candidate sums stacked in rank order, [world_size, C, K] binary64 -- the
    layout pwlq_search_finish adds up in a fixed order.  (An all-reduce would leave the order of
    the additions to the backend; K doubles per row make the gather just as cheap.)"""
    import torch
    parts = [torch.empty_like(sums_local) for _ in range(world_size)]
    dist.all_gather(parts, sums_local.contiguous(), group=group)
    return torch.stack(parts, dim=0)
