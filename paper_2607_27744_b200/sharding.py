"""Host-side sharding of a request-candidate batch across GPUs.

A request and all of its candidates form an independent unit (the GLM invariant, Eq. 1, and the
sharing identity, Eq. 11): no candidate output depends on another request.  The batch therefore
shards by REQUEST with no collective on the data path; weights are replicated.  Requests are
assigned greedily, heaviest first, to the least-loaded rank (longest-processing-time rule) under a
cost model of the three kernels; each rank then builds its own ``cand_offsets`` / ``seq_offsets``.
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import numpy as np


def request_cost(cand_counts: np.ndarray, seq_lens: Optional[np.ndarray] = None, c_linear: float = 1.0,
                 c_attn: float = 0.0, c_glm: float = 0.0) -> np.ndarray:
    """Relative cost of each request: n_r * (c_linear + c_glm + c_attn * L_r)."""
    n = np.asarray(cand_counts, np.float64)
    per_cand = c_linear + c_glm
    if seq_lens is not None and c_attn:
        per_cand = per_cand + c_attn * np.asarray(seq_lens, np.float64)
    return n * per_cand


def partition_requests(cost: Sequence[float], world_size: int) -> List[np.ndarray]:
    """Greedy longest-processing-time partition.  Returns, per rank, the sorted request indices."""
    cost = np.asarray(cost, np.float64)
    order = np.argsort(-cost, kind="stable")
    load = np.zeros(world_size)
    buckets: List[list] = [[] for _ in range(world_size)]
    for r in order:
        k = int(np.argmin(load))
        buckets[k].append(int(r))
        load[k] += cost[r]
    return [np.array(sorted(b), np.int64) for b in buckets]


def shard_rows(offsets: np.ndarray, requests: np.ndarray):
    """Rows (candidates or sequence positions) owned by `requests`, in request order, and the
    shard's own offsets array."""
    offsets = np.asarray(offsets, np.int64)
    counts = offsets[1:] - offsets[:-1]
    local = np.zeros(len(requests) + 1, np.int64)
    np.cumsum(counts[requests], out=local[1:])
    rows = np.concatenate([np.arange(offsets[r], offsets[r + 1]) for r in requests]) if len(requests) else \
        np.zeros(0, np.int64)
    return rows, local.astype(np.int32)


def replicate_offsets(offsets: np.ndarray, copies: int) -> np.ndarray:
    """Offsets of a global batch made of `copies` batches with these offsets, one after the other."""
    counts = np.diff(np.asarray(offsets, np.int64))
    out = np.zeros(copies * counts.size + 1, np.int64)
    np.cumsum(np.tile(counts, copies), out=out[1:])
    return out


class Shard:
    """What one rank scores of a global batch: its requests (global indices, ascending), the global
    candidate rows they own (in request order), the rank's own ``cand_offsets``, and the same for the
    sequence positions when the batch has sequences."""

    def __init__(self, requests, cand_rows, cand_offsets, seq_rows=None, seq_offsets=None):
        self.requests, self.cand_rows, self.cand_offsets = requests, cand_rows, cand_offsets
        self.seq_rows, self.seq_offsets = seq_rows, seq_offsets


def shard_batch(cand_offsets: np.ndarray, world_size: int, rank: int, seq_offsets: Optional[np.ndarray] = None,
                c_linear: float = 1.0, c_attn: float = 0.0, c_glm: float = 0.0) -> Shard:
    """Shard of `rank` when the global batch is split by request over `world_size` ranks (no rank
    needs anything from another: there is no collective on the data path)."""
    cand_offsets = np.asarray(cand_offsets, np.int64)
    lens = None if seq_offsets is None else np.diff(np.asarray(seq_offsets, np.int64))
    cost = request_cost(np.diff(cand_offsets), lens, c_linear=c_linear, c_attn=c_attn, c_glm=c_glm)
    mine = partition_requests(cost, world_size)[rank]
    rows, co_l = shard_rows(cand_offsets, mine)
    if seq_offsets is None:
        return Shard(mine, rows, co_l)
    seq_rows, so_l = shard_rows(seq_offsets, mine)
    return Shard(mine, rows, co_l, seq_rows, so_l)
