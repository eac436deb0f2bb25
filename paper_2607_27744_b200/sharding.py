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
    """What one rank scores of a global batch: its requests (global indices, ascending; a request that
    was split appears on several ranks), the global candidate rows they own (in request order), the
    rank's own ``cand_offsets``, and the same for the sequence positions when the batch has sequences."""

    def __init__(self, requests, cand_rows, cand_offsets, seq_rows=None, seq_offsets=None):
        self.requests, self.cand_rows, self.cand_offsets = requests, cand_rows, cand_offsets
        self.seq_rows, self.seq_offsets = seq_rows, seq_offsets


def split_requests(cand_offsets: np.ndarray, max_candidates: int):
    """Pieces of at most `max_candidates` consecutive candidates of one request: (request, first
    candidate row, count) per piece, in batch order.  A request with no candidates is one empty piece."""
    cand_offsets = np.asarray(cand_offsets, np.int64)
    req, start, count = [], [], []
    for r in range(cand_offsets.size - 1):
        a, b = int(cand_offsets[r]), int(cand_offsets[r + 1])
        if b == a:
            req.append(r), start.append(a), count.append(0)
        for c in range(a, b, max_candidates):
            req.append(r), start.append(c), count.append(min(max_candidates, b - c))
    return np.array(req, np.int64), np.array(start, np.int64), np.array(count, np.int64)


def shard_batch(cand_offsets: np.ndarray, world_size: int, rank: int, seq_offsets: Optional[np.ndarray] = None,
                c_linear: float = 1.0, c_attn: float = 0.0, c_glm: float = 0.0,
                max_share: Optional[float] = None) -> Shard:
    """Shard of `rank` when the global batch is split by request over `world_size` ranks (no rank
    needs anything from another: there is no collective on the data path).

    max_share: if given, a request whose cost exceeds this fraction of a rank's fair share is cut into
    pieces of consecutive candidates that may go to different ranks; each of those ranks then holds a
    copy of the request's own tensors (its row of X^R, its K and V), which is all a candidate needs from
    its request (Eq. 1).  Pieces of one request that land on the same rank are joined again."""
    cand_offsets = np.asarray(cand_offsets, np.int64)
    counts = np.diff(cand_offsets)
    lens = None if seq_offsets is None else np.diff(np.asarray(seq_offsets, np.int64))
    if max_share is None:
        cost = request_cost(counts, lens, c_linear=c_linear, c_attn=c_attn, c_glm=c_glm)
        mine = partition_requests(cost, world_size)[rank]
        rows, co_l = shard_rows(cand_offsets, mine)
        if seq_offsets is None:
            return Shard(mine, rows, co_l)
        seq_rows, so_l = shard_rows(seq_offsets, mine)
        return Shard(mine, rows, co_l, seq_rows, so_l)
    per_cand = request_cost(np.ones_like(counts), lens, c_linear=c_linear, c_attn=c_attn, c_glm=c_glm)
    fair = float((per_cand * counts).sum()) / world_size
    # the largest piece a request may keep, in candidates, from the cost of its candidates
    limit = np.maximum(1, np.floor(max_share * fair / np.maximum(per_cand, 1e-30))).astype(np.int64)
    req, start, count = [], [], []
    for r in range(counts.size):
        pr, ps, pc = split_requests(cand_offsets[r:r + 2], int(limit[r]))
        req.append(pr + r), start.append(ps), count.append(pc)
    req, start, count = np.concatenate(req), np.concatenate(start), np.concatenate(count)
    pieces = partition_requests(per_cand[req] * count, world_size)[rank]   # ascending: batch order
    # join pieces of the same request that are neighbours in the batch
    m_req, m_start, m_count = [], [], []
    for i in pieces:
        if m_req and m_req[-1] == req[i] and m_start[-1] + m_count[-1] == start[i]:
            m_count[-1] += int(count[i])
        else:
            m_req.append(int(req[i])), m_start.append(int(start[i])), m_count.append(int(count[i]))
    mine = np.array(m_req, np.int64)
    co_l = np.zeros(mine.size + 1, np.int64)
    np.cumsum(np.array(m_count, np.int64), out=co_l[1:])
    rows = np.concatenate([np.arange(a, a + c) for a, c in zip(m_start, m_count)]) if mine.size else np.zeros(0, np.int64)
    if seq_offsets is None:
        return Shard(mine, rows, co_l.astype(np.int32))
    seq_rows, so_l = shard_rows(seq_offsets, mine)
    return Shard(mine, rows, co_l.astype(np.int32), seq_rows, so_l)
