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
