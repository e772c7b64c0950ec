"""Host-side sharding of one pairwise matrix over ranks (one process per GPU).

Pairs are independent, so the unordered-pair index range of roomie_pair_matrix is cut into one
contiguous piece per rank, balanced by the walk cost of each pair (q_a + q_b path steps at most).
Every rank fills the entries of its own pairs in a zeroed matrix; since the pieces are disjoint,
a sum all-reduce (at most P*P*4 bytes, 1 MB for 512 profiles) is the gather.  No other data moves
between ranks: the library (a few tens of MB) is built on every rank from the same kernel table.
This module holds no kernel work and does not need a GPU."""
from __future__ import annotations

import numpy as np


def partition_pairs(offsets, world_size: int):
    """[(pair_begin, pair_end)] per rank: contiguous ranges of the row-major upper triangle
    (diagonal included) with near-equal sums of q_a + q_b."""
    q = np.diff(np.asarray(offsets, dtype=np.int64))
    P = len(q)
    a, b = np.triu_indices(P)
    cost = np.cumsum(q[a] + q[b])
    total = int(cost[-1]) if len(cost) else 0
    cuts = [0]
    for r in range(1, world_size):
        cuts.append(int(np.searchsorted(cost, total * r / world_size, side="left")))
    cuts.append(len(cost))
    cuts = np.maximum.accumulate(np.asarray(cuts))
    return [(int(cuts[r]), int(cuts[r + 1])) for r in range(world_size)]


def combine_shards(matrix, evals=None, group=None):
    """Sum all-reduce of the per-rank matrices (disjoint entries) and evaluation counts, in place.
    `matrix` / `evals` are torch tensors on the device the process group works on."""
    import torch.distributed as dist
    dist.all_reduce(matrix, op=dist.ReduceOp.SUM, group=group)
    if evals is not None:
        dist.all_reduce(evals, op=dist.ReduceOp.SUM, group=group)
    return matrix, evals


def pair_matrix_sharded(lib, rank: int, world_size: int, group=None, **kw):
    """Rank `rank`'s share of roomie_pair_matrix followed by the combine step.  Returns the full
    matrix and evaluation count on every rank."""
    from . import roomie
    lo, hi = partition_pairs(lib.offsets_host, world_size)[rank]
    out, evals = roomie.pair_matrix(lib, pair_begin=lo, pair_end=hi, **kw)
    return combine_shards(out, evals, group)
