"""ctypes binding of ``librocs.so`` (declared in ``include/rocs.h``).

Argument marshalling only: torch supplies device memory and streams, every step of the
computation runs inside the library's CUDA kernels.  There is no CPU or eager fallback: if the
library is missing or a call fails, an exception is raised.

Functions mirror the C entry points (``rocs_`` prefix dropped): :func:`plan_create`,
:func:`ikbo_linear`, :func:`linear`, :func:`dca_attention`, :func:`glm_interaction`.
bf16 tensors are ``torch.bfloat16``, fp32 tensors ``torch.float32``.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "librocs.so")
_lib = None

OK = 0
BF16, F32 = 0, 1
ACT_NONE, ACT_RELU = 0, 1
PATH_AUTO, PATH_GENERAL = 0, 1
NORM_LAYER, NORM_RMS = 0, 1

EXPORTS = [
    "rocs_status_string", "rocs_padded_ld", "rocs_set_path", "rocs_plan_create", "rocs_plan_destroy",
    "rocs_ikbo_linear_workspace", "rocs_ikbo_linear", "rocs_linear", "rocs_dca_attention_workspace",
    "rocs_dca_attention", "rocs_glm_interaction_workspace", "rocs_glm_interaction",
    "rocs_glm_fm_projection_workspace", "rocs_glm_fm_projection", "rocs_group_norm",
    "rocs_last_device_status", "rocs_ikbo_linear_static", "rocs_ikbo_linear_static_max_z_elems",
    "rocs_ikbo_linear_static_max_candidates", "rocs_ikbo_linear_stats_workspace", "rocs_ikbo_linear_stats",
    "rocs_weight_row_sums", "rocs_linear_normed",
]


class RocsError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} ({code})")


def lib() -> ctypes.CDLL:
    """Loads librocs.so on first use; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2607_27744_b200.build` "
                "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, i64, f32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_float, ctypes.c_size_t
        L.rocs_status_string.restype = ctypes.c_char_p
        L.rocs_status_string.argtypes = [ctypes.c_int]
        L.rocs_padded_ld.restype = i64
        L.rocs_padded_ld.argtypes = [i64, ctypes.c_int]
        L.rocs_set_path.argtypes = [ctypes.c_int]
        L.rocs_plan_create.argtypes = [ctypes.POINTER(vp), i32, i64, vp, vp, vp]
        L.rocs_plan_destroy.argtypes = [vp]
        L.rocs_ikbo_linear_workspace.restype = sz
        L.rocs_ikbo_linear_workspace.argtypes = [vp, i32]
        L.rocs_ikbo_linear.argtypes = [vp, ctypes.c_int, i32, i32, i32, vp, i64, vp, i64, vp, i64, vp, i64,
                                       vp, ctypes.c_int, vp, i64, vp, sz, vp]
        L.rocs_linear.argtypes = [ctypes.c_int, i64, i32, i32, vp, i64, vp, i64, vp, ctypes.c_int, vp, i64, vp]
        L.rocs_dca_attention_workspace.restype = sz
        L.rocs_dca_attention_workspace.argtypes = [vp, i32, i32, i32]
        L.rocs_dca_attention.argtypes = [vp, ctypes.c_int, i32, i32, i32, f32, vp, vp, vp, i64, vp, vp, vp, sz, vp]
        L.rocs_glm_interaction_workspace.restype = sz
        L.rocs_glm_interaction_workspace.argtypes = [vp, i32, i32, i32]
        L.rocs_glm_interaction.argtypes = [vp, ctypes.c_int, i32, i32, i32, vp, vp, vp, i32, i32, vp, vp, vp, vp,
                                           vp, sz, vp]
        L.rocs_glm_fm_projection_workspace.restype = sz
        L.rocs_glm_fm_projection_workspace.argtypes = [vp, i32, i32]
        L.rocs_glm_fm_projection.argtypes = [vp, ctypes.c_int, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp, sz, vp]
        L.rocs_group_norm.argtypes = [ctypes.c_int, ctypes.c_int, i64, i32, vp, i64, vp, vp, f32, vp, i64, vp]
        L.rocs_last_device_status.argtypes = [ctypes.POINTER(ctypes.c_uint32)]
        L.rocs_ikbo_linear_stats_workspace.restype = sz
        L.rocs_ikbo_linear_stats_workspace.argtypes = [vp, i32]
        L.rocs_ikbo_linear_stats.argtypes = [vp, ctypes.c_int, i32, i32, i32, vp, i64, vp, i64, vp, i64, vp, i64,
                                             vp, ctypes.c_int, vp, i64, vp, vp, sz, vp]
        L.rocs_weight_row_sums.argtypes = [ctypes.c_int, i32, i32, vp, i64, vp, vp]
        L.rocs_linear_normed.argtypes = [ctypes.c_int, ctypes.c_int, i64, i32, i32, vp, i64, vp, f32, vp, i64, vp, vp,
                                         ctypes.c_int, vp, i64, vp]
        L.rocs_ikbo_linear_static_max_z_elems.restype = sz
        L.rocs_ikbo_linear_static_max_candidates.restype = sz
        L.rocs_ikbo_linear_static.argtypes = [ctypes.c_int, i32, i64, vp, i32, i32, i32, vp, i64, vp, i64, vp, i64,
                                              vp, i64, vp, ctypes.c_int, vp, i64, vp]
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().rocs_status_string(code).decode()


def _check(code: int, where: str):
    if code != OK:
        raise RocsError(code, where)


def padded_ld(n: int, dtype: int) -> int:
    return int(lib().rocs_padded_ld(n, dtype))


def set_path(path: int):
    _check(lib().rocs_set_path(path), "rocs_set_path")


def last_device_status() -> int:
    """Synchronises, then raises RocsError if a bounded device-side wait expired."""
    detail = ctypes.c_uint32(0)
    code = lib().rocs_last_device_status(ctypes.byref(detail))
    if code != OK:
        raise RocsError(code, f"device status word 0x{detail.value:08x}")
    return detail.value


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return BF16
    if t.dtype == torch.float32:
        return F32
    raise TypeError(f"unsupported dtype {t.dtype}")


def _p(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream() -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _rows_2d(t: torch.Tensor):
    assert t.dim() == 2 and t.stride(1) == 1 and t.is_cuda, "expect a row-major 2-D CUDA tensor"
    return t.stride(0) if t.shape[0] > 1 else max(t.stride(0), t.shape[1])


class Plan:
    """Owns a ``rocs_plan_t`` (Section 4.1: the request-candidate map in segment form)."""

    def __init__(self, cand_offsets: torch.Tensor, cand_offsets_host=None):
        assert cand_offsets.is_cuda and cand_offsets.dtype == torch.int32 and cand_offsets.is_contiguous()
        self.cand_offsets = cand_offsets
        self.R = cand_offsets.numel() - 1
        if cand_offsets_host is None:
            host = cand_offsets.cpu()
        else:
            host = torch.as_tensor(cand_offsets_host, dtype=torch.int32).contiguous()
        self._host = host
        self.N = int(host[-1]) if host.numel() else 0
        handle = ctypes.c_void_p()
        _check(lib().rocs_plan_create(ctypes.byref(handle), self.R, self.N, _p(cand_offsets),
                                      ctypes.c_void_p(host.data_ptr()), _stream()), "rocs_plan_create")
        self.handle = handle

    def close(self):
        if getattr(self, "handle", None):
            lib().rocs_plan_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def plan_create(cand_offsets: torch.Tensor, cand_offsets_host=None) -> Plan:
    return Plan(cand_offsets, cand_offsets_host)


def ikbo_linear_workspace(plan: Plan, d_out: int) -> int:
    return int(lib().rocs_ikbo_linear_workspace(plan.handle, d_out))


def ikbo_linear(plan: Plan, XR: Optional[torch.Tensor], XC: torch.Tensor, W_CR: Optional[torch.Tensor],
                W_CC: torch.Tensor, bias: Optional[torch.Tensor] = None, relu: bool = False,
                out: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Y_i = act(Z[m_i] + X^C_i W_CC^T), Z = X^R W_CR^T + bias (Eq. 14).  W_CR / W_CC may be column
    slices of one [d_out, d_req + d_cand] weight."""
    d_req = 0 if XR is None else XR.shape[1]
    d_cand, d_out = XC.shape[1], W_CC.shape[0]
    assert XC.shape[0] == plan.N
    if out is None:
        out = torch.empty((plan.N, d_out), dtype=XC.dtype, device=XC.device)
    need = ikbo_linear_workspace(plan, d_out) if d_req > 0 else 0
    if need and workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=XC.device)
    if bias is not None:
        assert bias.dtype == torch.float32 and bias.is_contiguous()
    code = lib().rocs_ikbo_linear(
        plan.handle, _dtype_code(XC), d_req, d_cand, d_out,
        _p(XR), _rows_2d(XR) if d_req else 0, _p(XC), _rows_2d(XC),
        _p(W_CR) if d_req else None, _rows_2d(W_CR) if d_req else 0, _p(W_CC), _rows_2d(W_CC),
        _p(bias), ACT_RELU if relu else ACT_NONE, _p(out), _rows_2d(out),
        _p(workspace), workspace.numel() if workspace is not None else 0, _stream())
    _check(code, "rocs_ikbo_linear")
    return out


def ikbo_linear_stats(plan: Plan, XR: torch.Tensor, XC: torch.Tensor, W_CR: torch.Tensor, W_CC: torch.Tensor,
                      bias: Optional[torch.Tensor] = None, relu: bool = False, out: Optional[torch.Tensor] = None,
                      row_stats: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None):
    """ikbo_linear that also leaves each output row's (sum, sum of squares) for a normalisation folded
    into the next layer (Eq. 7).  Returns (Y, row_stats [N, 2] fp32)."""
    d_req, d_cand, d_out = XR.shape[1], XC.shape[1], W_CC.shape[0]
    assert XC.shape[0] == plan.N
    if out is None:
        out = torch.empty((plan.N, d_out), dtype=XC.dtype, device=XC.device)
    if row_stats is None:
        row_stats = torch.empty((plan.N, 2), dtype=torch.float32, device=XC.device)
    need = int(lib().rocs_ikbo_linear_stats_workspace(plan.handle, d_out))
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=XC.device)
    code = lib().rocs_ikbo_linear_stats(
        plan.handle, _dtype_code(XC), d_req, d_cand, d_out, _p(XR), _rows_2d(XR), _p(XC), _rows_2d(XC),
        _p(W_CR), _rows_2d(W_CR), _p(W_CC), _rows_2d(W_CC), _p(bias), ACT_RELU if relu else ACT_NONE, _p(out),
        _rows_2d(out), _p(row_stats), _p(workspace), workspace.numel(), _stream())
    _check(code, "rocs_ikbo_linear_stats")
    return out, row_stats


def weight_row_sums(W: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """wbar[n] = sum_k W[n, k] in fp32: the W 1 term of a LayerNorm folded into the layer."""
    d_out, d_in = W.shape
    if out is None:
        out = torch.empty(d_out, dtype=torch.float32, device=W.device)
    _check(lib().rocs_weight_row_sums(_dtype_code(W), d_out, d_in, _p(W), _rows_2d(W), _p(out), _stream()),
           "rocs_weight_row_sums")
    return out


def linear_normed(X: torch.Tensor, row_stats: torch.Tensor, W: torch.Tensor, wbar: Optional[torch.Tensor] = None,
                  bias: Optional[torch.Tensor] = None, eps: float = 1e-5, kind: int = NORM_LAYER, relu: bool = False,
                  out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Y = act(norm(X) W^T + bias) with the normalisation applied to the layer's accumulators (Eq. 7
    folded into the epilogue); gamma and beta are folded into W and bias by the caller."""
    M, d_in = X.shape
    d_out = W.shape[0]
    assert row_stats.dtype == torch.float32 and row_stats.shape == (M, 2) and row_stats.is_contiguous()
    if out is None:
        out = torch.empty((M, d_out), dtype=X.dtype, device=X.device)
    code = lib().rocs_linear_normed(_dtype_code(X), kind, M, d_in, d_out, _p(X), _rows_2d(X), _p(row_stats), float(eps),
                                    _p(W), _rows_2d(W), _p(wbar), _p(bias), ACT_RELU if relu else ACT_NONE, _p(out),
                                    _rows_2d(out), _stream())
    _check(code, "rocs_linear_normed")
    return out


def linear(X: torch.Tensor, W: torch.Tensor, bias: Optional[torch.Tensor] = None, relu: bool = False,
           out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Y = act(X W^T + bias), the one-group case of Eq. 4."""
    M, d_in = X.shape
    d_out = W.shape[0]
    if out is None:
        out = torch.empty((M, d_out), dtype=X.dtype, device=X.device)
    code = lib().rocs_linear(_dtype_code(X), M, d_in, d_out, _p(X), _rows_2d(X), _p(W), _rows_2d(W), _p(bias),
                             ACT_RELU if relu else ACT_NONE, _p(out), _rows_2d(out), _stream())
    _check(code, "rocs_linear")
    return out


def dca_attention(plan: Plan, Q: torch.Tensor, K: torch.Tensor, V: torch.Tensor, seq_offsets: torch.Tensor,
                  scale: float = 0.0, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Candidate-side cross attention over the request's shared K/V (Eq. 13).
    Q [N, n_q, H, dh]; K, V [T, H, dh]; seq_offsets int32 [R+1] on the device."""
    N, n_q, H, dh = Q.shape
    assert N == plan.N and Q.is_contiguous() and K.is_contiguous() and V.is_contiguous()
    assert seq_offsets.dtype == torch.int32 and seq_offsets.is_cuda and seq_offsets.numel() == plan.R + 1
    if out is None:
        out = torch.empty_like(Q)
    need = int(lib().rocs_dca_attention_workspace(plan.handle, n_q, H, dh))
    ws = torch.empty(need, dtype=torch.uint8, device=Q.device) if need else None
    code = lib().rocs_dca_attention(plan.handle, _dtype_code(Q), n_q, H, dh, float(scale), _p(Q), _p(K), _p(V),
                                    K.shape[0], _p(seq_offsets), _p(out), _p(ws), need, _stream())
    _check(code, "rocs_dca_attention")
    return out


def glm_interaction_workspace(plan: Plan, n_r: int, n_c: int, n_co: int) -> int:
    return int(lib().rocs_glm_interaction_workspace(plan.handle, n_r, n_c, n_co))


def glm_interaction(plan: Plan, XR: torch.Tensor, XC: torch.Tensor, W: Optional[torch.Tensor] = None,
                    n_ro: int = 0, n_co: int = 0, want_raw: bool = True, want_request_side: bool = True,
                    workspace: Optional[torch.Tensor] = None, outs: Optional[dict] = None) -> dict:
    """GLM factorization machine (Eq. 9-10) with optional row-axis compression (Eq. 5-6).
    Returns a dict with the tensors that were requested among YR, YC, OR, OC."""
    R, n_r, d = XR.shape
    N, n_c, _ = XC.shape
    n = n_r + n_c
    assert R == plan.R and N == plan.N and XR.is_contiguous() and XC.is_contiguous()
    dev, dt = XC.device, XC.dtype
    outs = dict(outs or {})
    if want_raw:
        if want_request_side:
            outs.setdefault("YR", torch.empty((R, n_r, n), dtype=dt, device=dev))
        outs.setdefault("YC", torch.empty((N, n_c, n), dtype=dt, device=dev))
    if W is not None:
        assert W.shape == (n_ro + n_co, n) and W.is_contiguous()
        if want_request_side:
            outs.setdefault("OR", torch.empty((R, n_ro, n), dtype=dt, device=dev))
        outs.setdefault("OC", torch.empty((N, n_co, n), dtype=dt, device=dev))
    need = glm_interaction_workspace(plan, n_r, n_c, n_co) if W is not None else 0
    if need and workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=dev)
    code = lib().rocs_glm_interaction(
        plan.handle, _dtype_code(XC), n_r, n_c, d, _p(XR), _p(XC), _p(W), n_ro, n_co,
        _p(outs.get("YR")), _p(outs.get("YC")), _p(outs.get("OR")), _p(outs.get("OC")),
        _p(workspace), workspace.numel() if workspace is not None else 0, _stream())
    _check(code, "rocs_glm_interaction")
    return outs


def glm_fm_projection_workspace(plan: Plan, d: int, k: int) -> int:
    return int(lib().rocs_glm_fm_projection_workspace(plan.handle, d, k))


def glm_fm_projection(plan: Plan, XR: torch.Tensor, XC: torch.Tensor, P: torch.Tensor,
                      want_request_side: bool = True, workspace: Optional[torch.Tensor] = None,
                      outs: Optional[dict] = None) -> dict:
    """GLM factorization machine (Eq. 9-10) projected to k columns, F = G P with P [n_r + n_c, k].
    Returns a dict with FC [N, n_c, k] and, if requested, FR [R, n_r, k]."""
    R, n_r, d = XR.shape
    N, n_c, _ = XC.shape
    k = P.shape[1]
    assert R == plan.R and N == plan.N and XR.is_contiguous() and XC.is_contiguous()
    assert P.shape[0] == n_r + n_c and P.is_contiguous() and P.dtype == XC.dtype
    dev, dt = XC.device, XC.dtype
    outs = dict(outs or {})
    if want_request_side:
        outs.setdefault("FR", torch.empty((R, n_r, k), dtype=dt, device=dev))
    outs.setdefault("FC", torch.empty((N, n_c, k), dtype=dt, device=dev))
    need = glm_fm_projection_workspace(plan, d, k)
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=dev)
    code = lib().rocs_glm_fm_projection(
        plan.handle, _dtype_code(XC), n_r, n_c, d, k, _p(XR), _p(XC), _p(P), _p(outs.get("FR")), _p(outs.get("FC")),
        _p(workspace), workspace.numel(), _stream())
    _check(code, "rocs_glm_fm_projection")
    return outs


def group_norm(X: torch.Tensor, gamma: Optional[torch.Tensor] = None, beta: Optional[torch.Tensor] = None,
               eps: float = 1e-5, kind: int = NORM_LAYER, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Group-local LayerNorm / RMSNorm (Eq. 7) of one group's tensor X [M, d], row by row."""
    assert X.dim() == 2 and X.stride(1) == 1
    M, d = X.shape
    if out is None:
        out = torch.empty((M, d), dtype=X.dtype, device=X.device)
    code = lib().rocs_group_norm(_dtype_code(X), kind, M, d, _p(X), _rows_2d(X), _p(gamma), _p(beta), eps, _p(out),
                                 _rows_2d(out), _stream())
    _check(code, "rocs_group_norm")
    return out


def ikbo_linear_static(cand_offsets: torch.Tensor, XR: torch.Tensor, XC: torch.Tensor, W_CR: torch.Tensor,
                       W_CC: torch.Tensor, out: torch.Tensor, bias: Optional[torch.Tensor] = None,
                       relu: bool = False) -> torch.Tensor:
    """The split linear layer through ``rocs_ikbo_linear_static``: no plan, no workspace, and the call
    allocates nothing -- for hosts that cannot call cudaMalloc while scoring.  The caller passes the
    output tensor; scratch lives in a fixed array inside the library (limits: R * d_out <= 1 Mi,
    N <= 256 Ki; calls share the array, so do not let two of them overlap on the GPU)."""
    R, N = cand_offsets.numel() - 1, XC.shape[0]
    code = lib().rocs_ikbo_linear_static(
        _dtype_code(XC), R, N, _p(cand_offsets), XR.shape[1], XC.shape[1], W_CC.shape[0], _p(XR), _rows_2d(XR),
        _p(XC), _rows_2d(XC), _p(W_CR), _rows_2d(W_CR), _p(W_CC), _rows_2d(W_CC), _p(bias),
        ACT_RELU if relu else ACT_NONE, _p(out), _rows_2d(out), _stream())
    _check(code, "rocs_ikbo_linear_static")
    return out
