"""ctypes front end of the fp64 CPU oracle (``rocs_ref.c``).

TEST INFRASTRUCTURE, NOT THE PRODUCT: only the tests, the smoke check and the
benchmark's cpu_baseline / reference legs import this module.  It never touches
the CUDA library and the CUDA binding never touches it.

Arrays are numpy.  Storage types: bf16 is carried as ``uint16`` bit patterns,
fp32 as ``float32``, fp64 as ``float64``; every result is ``float64``.
Each wrapper names the passage of the paper its C function follows.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "rocs_ref.c")
_SO = os.path.join(_HERE, "librocs_ref.so")
_lib = None

_DT = {np.dtype(np.uint16): 0, np.dtype(np.float32): 1, np.dtype(np.float64): 2}


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP).  Returns the library path."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", _SO, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _SO


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.rocs_ref_num_threads.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(_load().rocs_ref_num_threads())


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _same_dtype(*arrays):
    dts = {a.dtype for a in arrays if a is not None}
    assert len(dts) == 1, f"mixed storage types {dts}"
    dt = dts.pop()
    assert dt in _DT, f"unsupported storage type {dt}"
    return _DT[dt]


def _c(a, dtype=None):
    if a is None:
        return None
    a = np.ascontiguousarray(a)
    return a if dtype is None else a.astype(dtype, copy=False)


def _offsets(o):
    o = np.ascontiguousarray(o, dtype=np.int32)
    assert o.ndim == 1 and o[0] == 0 and np.all(np.diff(o) >= 0)
    return o


def _sample(sample):
    if sample is None:
        return None, 0
    s = np.ascontiguousarray(sample, dtype=np.int64)
    return s, s.size


def ikbo_linear(cand_offsets, XR, XC, W, bias=None, relu=False, sample=None):
    """Eq. 4 (two groups) in materialised form.  W is [d_out, d_req + d_cand]."""
    co = _offsets(cand_offsets)
    R, N = co.size - 1, int(co[-1])
    XR, XC, W = _c(XR), _c(XC), _c(W)
    d_req = XR.shape[1] if XR is not None and XR.size else 0
    d_cand = XC.shape[1]
    d_out = W.shape[0]
    assert W.shape[1] == d_req + d_cand and XC.shape[0] == N
    if d_req == 0:
        XR = np.zeros((R, 0), XC.dtype)
    dt = _same_dtype(XR, XC, W)
    b = _c(bias, np.float64)
    s, ns = _sample(sample)
    Y = np.empty((ns if s is not None else N, d_out), np.float64)
    rc = _load().rocs_ref_ikbo_linear(
        dt, R, ctypes.c_int64(N), _ptr(co), d_req, d_cand, d_out, _ptr(XR), _ptr(XC), _ptr(W),
        _ptr(b), int(relu), _ptr(s), ctypes.c_int64(ns), _ptr(Y))
    assert rc == 0
    return Y


def ikbo_linear_decomposed(cand_offsets, XR, XC, W, bias=None, relu=False):
    """Section 4.1 + Eq. 14: Z once per request, then Y_i = Z[m_i] + W_CC x_i.  Returns (Z, Y)."""
    co = _offsets(cand_offsets)
    R, N = co.size - 1, int(co[-1])
    XR, XC, W = _c(XR), _c(XC), _c(W)
    d_req, d_cand, d_out = XR.shape[1], XC.shape[1], W.shape[0]
    dt = _same_dtype(XR, XC, W)
    b = _c(bias, np.float64)
    Z = np.empty((R, d_out), np.float64)
    Y = np.empty((N, d_out), np.float64)
    rc = _load().rocs_ref_ikbo_linear_decomposed(
        dt, R, ctypes.c_int64(N), _ptr(co), d_req, d_cand, d_out, _ptr(XR), _ptr(XC), _ptr(W),
        _ptr(b), int(relu), _ptr(Z), _ptr(Y))
    assert rc == 0
    return Z, Y


def dca_attention(cand_offsets, seq_offsets, Q, K, V, scale=None, sample=None):
    """Eq. 13, candidate side, on candidate-batched copies of K and V.

    Q [N, n_q, H, dh]; K, V [T, H, dh]; returns O [rows, n_q, H, dh] fp64."""
    co, so = _offsets(cand_offsets), _offsets(seq_offsets)
    R, N = co.size - 1, int(co[-1])
    Q, K, V = _c(Q), _c(K), _c(V)
    _, n_q, H, dh = Q.shape
    assert Q.shape[0] == N and K.shape == V.shape and K.shape[0] == int(so[-1]) and K.shape[1:] == (H, dh)
    dt = _same_dtype(Q, K, V)
    if scale is None:
        scale = 1.0 / np.sqrt(dh)
    s, ns = _sample(sample)
    O = np.empty((ns if s is not None else N, n_q, H, dh), np.float64)
    rc = _load().rocs_ref_dca_attention(
        dt, R, ctypes.c_int64(N), _ptr(co), _ptr(so), n_q, H, dh, ctypes.c_double(scale),
        _ptr(Q), _ptr(K), _ptr(V), _ptr(s), ctypes.c_int64(ns), _ptr(O))
    assert rc == 0
    return O


def dca_attention_shared(cand_offsets, seq_offsets, Q, K, V, scale=None):
    """Section 4.3.1: K/V indexed in place through the request map (no copies)."""
    co, so = _offsets(cand_offsets), _offsets(seq_offsets)
    R, N = co.size - 1, int(co[-1])
    Q, K, V = _c(Q), _c(K), _c(V)
    _, n_q, H, dh = Q.shape
    dt = _same_dtype(Q, K, V)
    if scale is None:
        scale = 1.0 / np.sqrt(dh)
    O = np.empty((N, n_q, H, dh), np.float64)
    rc = _load().rocs_ref_dca_attention_shared(
        dt, R, ctypes.c_int64(N), _ptr(co), _ptr(so), n_q, H, dh, ctypes.c_double(scale),
        _ptr(Q), _ptr(K), _ptr(V), _ptr(O))
    assert rc == 0
    return O


def glm_interaction(cand_offsets, XR, XC, W=None, n_ro=0, n_co=0, sample=None):
    """Eq. 9-10 on the materialised X = [X^R[m_i]; X^C[i]], then Eq. 5-6 if W is given.

    XR [R, n_r, d], XC [N, n_c, d], W [n_ro + n_co, n_r + n_c].
    Returns (G, O): G [rows, n, n] masked interaction (first n_r rows request side,
    last n_c rows candidate side), O [rows, n_ro + n_co, n] or None."""
    co = _offsets(cand_offsets)
    R, N = co.size - 1, int(co[-1])
    XR, XC, W = _c(XR), _c(XC), _c(W)
    n_r, d = XR.shape[1], XR.shape[2]
    n_c = XC.shape[1]
    n = n_r + n_c
    assert XC.shape[0] == N and XC.shape[2] == d
    dt = _same_dtype(XR, XC, W)
    s, ns = _sample(sample)
    rows = ns if s is not None else N
    G = np.empty((rows, n, n), np.float64)
    O = None
    if W is not None:
        assert W.shape == (n_ro + n_co, n)
        O = np.empty((rows, n_ro + n_co, n), np.float64)
    rc = _load().rocs_ref_glm_interaction(
        dt, R, ctypes.c_int64(N), _ptr(co), n_r, n_c, d, _ptr(XR), _ptr(XC), _ptr(W), n_ro, n_co,
        _ptr(s), ctypes.c_int64(ns), _ptr(G), _ptr(O))
    assert rc == 0
    return G, O


def glm_interaction_decomposed(cand_offsets, XR, XC, W=None, n_ro=0, n_co=0):
    """Request-once form: returns (YR [R,n_r,n], YC [N,n_c,n], OR [R,n_ro,n], OC [N,n_co,n])."""
    co = _offsets(cand_offsets)
    R, N = co.size - 1, int(co[-1])
    XR, XC, W = _c(XR), _c(XC), _c(W)
    n_r, d = XR.shape[1], XR.shape[2]
    n_c = XC.shape[1]
    n = n_r + n_c
    dt = _same_dtype(XR, XC, W)
    YR = np.empty((R, n_r, n), np.float64)
    YC = np.empty((N, n_c, n), np.float64)
    OR = OC = None
    if W is not None:
        OR = np.empty((R, n_ro, n), np.float64)
        OC = np.empty((N, n_co, n), np.float64)
    rc = _load().rocs_ref_glm_interaction_decomposed(
        dt, R, ctypes.c_int64(N), _ptr(co), n_r, n_c, d, _ptr(XR), _ptr(XC), _ptr(W), n_ro, n_co,
        _ptr(YR), _ptr(YC), _ptr(OR), _ptr(OC))
    assert rc == 0
    return YR, YC, OR, OC


def glm_fm_projection(cand_offsets, XR, XC, P, sample=None):
    """Eq. 9-10 on the materialised X = [X^R[m_i]; X^C[i]], then F = G P (P [n_r + n_c, k]).

    Returns F [rows, n, k]: first n_r rows request side, last n_c rows candidate side."""
    co = _offsets(cand_offsets)
    R, N = co.size - 1, int(co[-1])
    XR, XC, P = _c(XR), _c(XC), _c(P)
    n_r, d = XR.shape[1], XR.shape[2]
    n_c = XC.shape[1]
    n = n_r + n_c
    assert XC.shape[0] == N and XC.shape[2] == d and P.shape[0] == n
    k = P.shape[1]
    dt = _same_dtype(XR, XC, P)
    s, ns = _sample(sample)
    rows = ns if s is not None else N
    F = np.empty((rows, n, k), np.float64)
    rc = _load().rocs_ref_glm_fm_projection(
        dt, R, ctypes.c_int64(N), _ptr(co), n_r, n_c, d, k, _ptr(XR), _ptr(XC), _ptr(P),
        _ptr(s), ctypes.c_int64(ns), _ptr(F))
    assert rc == 0
    return F


def glm_fm_projection_decomposed(cand_offsets, XR, XC, P):
    """Request-once form: returns (FR [R, n_r, k], FC [N, n_c, k])."""
    co = _offsets(cand_offsets)
    R, N = co.size - 1, int(co[-1])
    XR, XC, P = _c(XR), _c(XC), _c(P)
    n_r, d = XR.shape[1], XR.shape[2]
    n_c = XC.shape[1]
    k = P.shape[1]
    dt = _same_dtype(XR, XC, P)
    FR = np.empty((R, n_r, k), np.float64)
    FC = np.empty((N, n_c, k), np.float64)
    rc = _load().rocs_ref_glm_fm_projection_decomposed(
        dt, R, ctypes.c_int64(N), _ptr(co), n_r, n_c, d, k, _ptr(XR), _ptr(XC), _ptr(P), _ptr(FR), _ptr(FC))
    assert rc == 0
    return FR, FC


LAYER_NORM, RMS_NORM = 0, 1


def group_norm(X, gamma=None, beta=None, eps=1e-5, kind=LAYER_NORM):
    """Eq. 7 on one group's tensor X [M, d]: LayerNorm (biased variance) or RMSNorm over each row."""
    X, gamma, beta = _c(X), _c(gamma), _c(beta)
    M, d = X.shape
    dt = _same_dtype(X, gamma, beta)
    Y = np.empty((M, d), np.float64)
    rc = _load().rocs_ref_group_norm(dt, ctypes.c_int64(M), d, _ptr(X), _ptr(gamma), _ptr(beta),
                                     ctypes.c_double(eps), kind, _ptr(Y))
    assert rc == 0
    return Y
