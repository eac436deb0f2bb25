"""Helpers shared by the GPU parity tests (marshalling and the error metric only)."""
import numpy as np
import torch

BF16_TOL = 1e-2   # max |gpu - ref| <= 1e-2 * max |ref|   (bf16 storage)
F32_TOL = 1e-4    # same normalisation, fp32 path


def to_dev(a):
    """numpy array from workloads (uint16 = bf16 bits, float32, int32) -> CUDA tensor."""
    if a is None:
        return None
    t = torch.from_numpy(np.ascontiguousarray(a))
    if a.dtype == np.uint16:
        t = t.view(torch.bfloat16)
    return t.cuda()


def to_host_f64(t):
    return t.detach().to(torch.float64).cpu().numpy()


def rel_err(got, ref):
    """max_i |got_i - ref_i| / max_i |ref_i| over one output tensor."""
    ref = np.asarray(ref, np.float64)
    got = np.asarray(got, np.float64)
    assert got.shape == ref.shape, (got.shape, ref.shape)
    if ref.size == 0:
        return 0.0
    assert np.all(np.isfinite(got)), "non-finite values in the GPU output"
    denom = np.abs(ref).max()
    return float(np.abs(got - ref).max() / (denom if denom > 0 else 1.0))


def tol_for(dtype):
    return BF16_TOL if dtype == "bf16" else F32_TOL
