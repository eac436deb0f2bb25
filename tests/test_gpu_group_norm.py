"""GPU parity of the group-local normalisation (Eq. 7) against the fp64 oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import rocs_ref as ref
from paper_2607_27744_b200 import binding as rocs, workloads as wl
from _util import rel_err, to_dev, to_host_f64, tol_for

pytestmark = pytest.mark.gpu


def _inputs(M, d, dtype, seed):
    x = wl.normal((M, d), 9, 70 + seed, dtype)
    gamma = wl.store(1.0 + 0.25 * wl.to_f64(wl.normal((d,), 9, 80 + seed, "f32")).astype(np.float32), dtype)
    beta = wl.normal((d,), 9, 90 + seed, dtype, std=0.5)
    return x, gamma, beta


@pytest.mark.parametrize("kind", [rocs.NORM_LAYER, rocs.NORM_RMS])
@pytest.mark.parametrize("dtype,d", [("bf16", 256), ("bf16", 1024), ("bf16", 768), ("bf16", 1536), ("bf16", 2048), ("bf16", 4096),
                                     ("bf16", 40), ("f32", 128), ("f32", 96), ("f32", 1024)])
def test_rows_against_the_oracle(kind, dtype, d):
    x, gamma, beta = _inputs(1237, d, dtype, d % 7)
    y = rocs.group_norm(to_dev(x), to_dev(gamma), to_dev(beta), eps=1e-5, kind=kind)
    want = ref.group_norm(x, gamma, beta, 1e-5, kind)
    assert rel_err(to_host_f64(y), want) <= tol_for(dtype)


def test_no_scale_no_shift_strided_rows_and_in_place():
    x, _, _ = _inputs(300, 512, "bf16", 3)
    buf = torch.zeros((300, 640), dtype=torch.bfloat16, device="cuda")
    buf[:, :512] = to_dev(x)
    view = buf[:, :512]                      # row stride 640
    want = ref.group_norm(x, None, None, 1e-6, ref.RMS_NORM)
    y = rocs.group_norm(view, eps=1e-6, kind=rocs.NORM_RMS)
    assert rel_err(to_host_f64(y), want) <= tol_for("bf16")
    rocs.group_norm(view, eps=1e-6, kind=rocs.NORM_RMS, out=view)   # Y aliases X
    assert rel_err(to_host_f64(view), want) <= tol_for("bf16")
    assert torch.all(buf[:, 512:] == 0)


def test_config2_activation_shape_sampled_and_rows_are_isolated():
    # the candidate-side activations of the retrieval MLP: 131072 x 1024
    M, d = 131072, 1024
    x, gamma, beta = _inputs(M, d, "bf16", 5)
    X = to_dev(x)
    y = rocs.group_norm(X, to_dev(gamma), to_dev(beta), kind=rocs.NORM_LAYER)
    sample = np.unique(np.concatenate([[0, M - 1], np.random.default_rng(2).integers(0, M, 500)]))
    want = ref.group_norm(x[sample], gamma, beta, 1e-5, ref.LAYER_NORM)
    assert rel_err(to_host_f64(y[torch.from_numpy(sample).cuda()]), want) <= tol_for("bf16")
    X2 = X.clone()
    X2[4321] += 1.0
    y2 = rocs.group_norm(X2, to_dev(gamma), to_dev(beta), kind=rocs.NORM_LAYER)
    same = (y.view(torch.int16) == y2.view(torch.int16)).all(dim=1)
    assert bool(same[:4321].all()) and bool(same[4322:].all()) and not bool(same[4321])


def test_empty_and_errors():
    _, gamma, beta = _inputs(1, 256, "bf16", 1)
    y = rocs.group_norm(torch.empty((0, 256), dtype=torch.bfloat16, device="cuda"), to_dev(gamma), to_dev(beta))
    assert y.shape == (0, 256)
    X = torch.zeros((4, 256), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(rocs.RocsError) as e:
        rocs.group_norm(X, kind=7)
    assert e.value.code == -1  # ROCS_ERR_INVALID_ARG
    with pytest.raises(rocs.RocsError) as e:
        rocs.group_norm(X, eps=-1.0)
    assert e.value.code == -1
