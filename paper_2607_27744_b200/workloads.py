"""Seeded synthetic inputs shaped like the paper's retrieval and ranking workloads.

This module only draws random numbers and lays them out; it contains none of the
method's arithmetic, so the CPU oracle's tests and the CUDA path's tests can both
feed from it without sharing any computation.

The paper's workloads are production traffic (ads retrieval with thousands of
candidates per request, ranking with hundreds, user histories of hundreds to
thousands of tokens; Section 4.3 and the end-to-end table of Section 5) and are
not available, so every tensor here is N(0, 1) (weights N(0, 1/fan_in) variance)
with the request/candidate structure of the five benchmark configurations:

  1 tiny fp32        R=4, 1..16 candidates per request
  2 retrieval MLP    R=256 x 512 candidates, 768->1024->1024->256, layer 1 split 512|256
  3 DCA ranking      R=64, lognormal(6.5, 0.8) candidates clipped to [1, 4096], L=2048, 8x64
  4 GLM Wukong       R=128 x 1024 candidates, 32 request + 16 candidate embeddings of dim 128
  5 skewed mixed     R=1024, Zipf(1.2) candidates clipped to [1, 8192], L in [256, 1024]

bf16 tensors are returned as uint16 bit patterns (drawn in fp32, rounded to nearest
even), fp32 tensors as float32; both sides of a parity test consume the same bits.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Optional

import numpy as np

SEED = (2607, 27744)
_CHUNK_ROWS = 1 << 16


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest even) and return the 16-bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def to_f64(a: np.ndarray) -> np.ndarray:
    """Exact widening of either storage type."""
    if a.dtype == np.uint16:
        return bf16_bits_to_f32(a).astype(np.float64)
    return a.astype(np.float64)


def store(x_f32: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == "bf16":
        return f32_to_bf16_bits(x_f32)
    assert dtype == "f32"
    return np.ascontiguousarray(x_f32, dtype=np.float32)


def _rng(cfg_id: int, stream: int, chunk: int = 0) -> np.random.Generator:
    return np.random.default_rng([*SEED, cfg_id, stream, chunk])


def normal(shape, cfg_id: int, stream: int, dtype: str, std: float = 1.0) -> np.ndarray:
    """N(0, std^2) tensor, generated in fixed row chunks so memory stays bounded."""
    shape = tuple(int(s) for s in shape)
    rows = shape[0]
    inner = int(np.prod(shape[1:], dtype=np.int64)) if len(shape) > 1 else 1
    out = np.empty((rows, inner), np.uint16 if dtype == "bf16" else np.float32)
    for c, r0 in enumerate(range(0, rows, _CHUNK_ROWS)):
        r1 = min(rows, r0 + _CHUNK_ROWS)
        x = _rng(cfg_id, stream, c).standard_normal((r1 - r0, inner), dtype=np.float32)
        if std != 1.0:
            x *= np.float32(std)
        out[r0:r1] = store(x, dtype)
    return out.reshape(shape)


def offsets_from_counts(counts) -> np.ndarray:
    counts = np.asarray(counts, dtype=np.int64)
    off = np.zeros(counts.size + 1, np.int64)
    np.cumsum(counts, out=off[1:])
    assert off[-1] < 2**31
    return off.astype(np.int32)


@dataclass(frozen=True)
class Config:
    cfg_id: int
    dtype: str
    R: int
    count_law: str            # "uniform16" | "const" | "lognormal" | "zipf"
    count_const: int = 0
    # linear
    d_req: int = 0
    d_cand: int = 0
    d_out: int = 0
    mlp_hidden: tuple = ()    # further plain layers after the split one
    # DCA
    L_law: str = "const"      # "const" | "uniform"
    L_const: int = 0
    L_lo: int = 0
    L_hi: int = 0
    H: int = 0
    dh: int = 0
    n_q: int = 1
    dca_layers: int = 0
    d_feat: int = 0           # candidate feature width feeding the query projection
    # GLM
    n_r: int = 0
    n_c: int = 0
    d_emb: int = 0
    n_ro: int = 0
    n_co: int = 0

    def with_(self, **kw) -> "Config":
        return replace(self, **kw)


CONFIGS = {
    1: Config(1, "f32", R=4, count_law="uniform16", d_req=64, d_cand=32, d_out=64,
              L_const=32, H=2, dh=32, dca_layers=1, d_feat=32, n_r=4, n_c=2, d_emb=16),
    2: Config(2, "bf16", R=256, count_law="const", count_const=512, d_req=512, d_cand=256,
              d_out=1024, mlp_hidden=(1024, 256)),
    3: Config(3, "bf16", R=64, count_law="lognormal", L_const=2048, H=8, dh=64, dca_layers=2,
              d_feat=512),
    4: Config(4, "bf16", R=128, count_law="const", count_const=1024, n_r=32, n_c=16, d_emb=128,
              n_ro=8, n_co=8),
    5: Config(5, "bf16", R=1024, count_law="zipf", d_req=768, d_cand=256, d_out=1024,
              L_law="uniform", L_lo=256, L_hi=1024, H=8, dh=64, dca_layers=1, n_r=24, n_c=8,
              d_emb=128),
}


def candidate_counts(cfg: Config) -> np.ndarray:
    g = _rng(cfg.cfg_id, 0)
    if cfg.count_law == "uniform16":
        return g.integers(1, 17, size=cfg.R)
    if cfg.count_law == "const":
        return np.full(cfg.R, cfg.count_const, np.int64)
    if cfg.count_law == "lognormal":
        return np.clip(np.rint(g.lognormal(6.5, 0.8, size=cfg.R)), 1, 4096).astype(np.int64)
    if cfg.count_law == "zipf":
        return np.clip(g.zipf(1.2, size=cfg.R), 1, 8192).astype(np.int64)
    raise ValueError(cfg.count_law)


def sequence_lengths(cfg: Config) -> np.ndarray:
    if cfg.L_law == "const":
        return np.full(cfg.R, cfg.L_const, np.int64)
    return _rng(cfg.cfg_id, 1).integers(cfg.L_lo, cfg.L_hi + 1, size=cfg.R)


def cand_offsets(cfg: Config) -> np.ndarray:
    return offsets_from_counts(candidate_counts(cfg))


def seq_offsets(cfg: Config) -> np.ndarray:
    return offsets_from_counts(sequence_lengths(cfg))


def linear_inputs(cfg: Config, co: Optional[np.ndarray] = None, bias: bool = False):
    """X^R [R, d_req], X^C [N, d_cand], W [d_out, d_req + d_cand] (= [W_CR | W_CC])."""
    co = cand_offsets(cfg) if co is None else co
    N = int(co[-1])
    fan_in = cfg.d_req + cfg.d_cand
    d = dict(
        cand_offsets=co,
        XR=normal((cfg.R, cfg.d_req), cfg.cfg_id, 10, cfg.dtype),
        XC=normal((N, cfg.d_cand), cfg.cfg_id, 11, cfg.dtype),
        W=normal((cfg.d_out, fan_in), cfg.cfg_id, 12, cfg.dtype, std=fan_in ** -0.5),
        bias=None,
    )
    if bias:
        d["bias"] = _rng(cfg.cfg_id, 13).standard_normal(cfg.d_out).astype(np.float32)
    return d


def mlp_weights(cfg: Config):
    """Weights of the plain layers that follow the split layer (config 2)."""
    ws, fan_in = [], cfg.d_out
    for li, width in enumerate(cfg.mlp_hidden):
        ws.append(normal((width, fan_in), cfg.cfg_id, 20 + li, cfg.dtype, std=fan_in ** -0.5))
        fan_in = width
    return ws


def dca_inputs(cfg: Config, co: Optional[np.ndarray] = None, so: Optional[np.ndarray] = None,
               layer: int = 0):
    """Q [N, n_q, H, dh] and the request's K, V [T, H, dh], all N(0, 1)."""
    co = cand_offsets(cfg) if co is None else co
    so = seq_offsets(cfg) if so is None else so
    N, T = int(co[-1]), int(so[-1])
    return dict(
        cand_offsets=co, seq_offsets=so,
        Q=normal((N, cfg.n_q, cfg.H, cfg.dh), cfg.cfg_id, 30 + 4 * layer, cfg.dtype),
        K=normal((T, cfg.H, cfg.dh), cfg.cfg_id, 31 + 4 * layer, cfg.dtype),
        V=normal((T, cfg.H, cfg.dh), cfg.cfg_id, 32 + 4 * layer, cfg.dtype),
    )


def dca_stack_inputs(cfg: Config, co: Optional[np.ndarray] = None, so: Optional[np.ndarray] = None):
    """Candidate features x^C [N, d_feat], per layer W_Q [H*dh, width of h_{l-1}], K_l, V_l."""
    co = cand_offsets(cfg) if co is None else co
    so = seq_offsets(cfg) if so is None else so
    N, T = int(co[-1]), int(so[-1])
    layers, width = [], cfg.d_feat
    for l in range(cfg.dca_layers):
        layers.append(dict(
            WQ=normal((cfg.H * cfg.dh, width), cfg.cfg_id, 40 + 4 * l, cfg.dtype, std=width ** -0.5),
            K=normal((T, cfg.H, cfg.dh), cfg.cfg_id, 41 + 4 * l, cfg.dtype),
            V=normal((T, cfg.H, cfg.dh), cfg.cfg_id, 42 + 4 * l, cfg.dtype),
        ))
        width += cfg.H * cfg.dh
    return dict(cand_offsets=co, seq_offsets=so,
                XC=normal((N, cfg.d_feat), cfg.cfg_id, 39, cfg.dtype), layers=layers)


def glm_inputs(cfg: Config, co: Optional[np.ndarray] = None):
    """X^R [R, n_r, d], X^C [N, n_c, d], compression W [n_ro + n_co, n_r + n_c] or None."""
    co = cand_offsets(cfg) if co is None else co
    N = int(co[-1])
    n = cfg.n_r + cfg.n_c
    W = None
    if cfg.n_ro + cfg.n_co > 0:
        W = normal((cfg.n_ro + cfg.n_co, n), cfg.cfg_id, 52, cfg.dtype, std=n ** -0.5)
    return dict(
        cand_offsets=co,
        XR=normal((cfg.R, cfg.n_r, cfg.d_emb), cfg.cfg_id, 50, cfg.dtype),
        XC=normal((N, cfg.n_c, cfg.d_emb), cfg.cfg_id, 51, cfg.dtype),
        W=W,
    )


def fm_projection_weight(cfg: Config, k: int) -> np.ndarray:
    """Projection P [n_r + n_c, k] of the interaction matrix's column axis, N(0, 1/n)."""
    n = cfg.n_r + cfg.n_c
    return normal((n, k), cfg.cfg_id, 53, cfg.dtype, std=n ** -0.5)


def stratified_sample(co: np.ndarray, n_uniform: int = 256, n_small_requests: int = 8,
                      whole_largest: bool = False, seed_stream: int = 90, cfg_id: int = 0) -> np.ndarray:
    """Candidate indices for sampled checks at full size: first and last candidate of every
    request, every candidate of the smallest requests, optionally one whole largest request,
    plus uniform draws."""
    co = np.asarray(co, np.int64)
    counts = np.diff(co)
    nz = np.nonzero(counts)[0]
    picks = [co[nz], co[nz + 1] - 1]
    order = nz[np.argsort(counts[nz], kind="stable")]
    for r in order[:n_small_requests]:
        picks.append(np.arange(co[r], co[r + 1]))
    if whole_largest and order.size:
        r = order[-1]
        picks.append(np.arange(co[r], co[r + 1]))
    N = int(co[-1])
    if N > 0 and n_uniform > 0:
        picks.append(_rng(cfg_id, seed_stream).integers(0, N, size=n_uniform))
    return np.unique(np.concatenate(picks)).astype(np.int64)
