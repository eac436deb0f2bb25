"""GPU parity of the projected factorization machine (F = G P on Eq. 9-10) against the fp64 oracle,
through the C ABI.  bf16: max |gpu - ref| <= 1e-2 max |ref|; fp32: 1e-4; isolation: bit-exact."""
import numpy as np
import pytest
import torch

from oracle import rocs_ref as ref
from paper_2607_27744_b200 import binding as rocs, workloads as wl
from _util import rel_err, to_dev, to_host_f64, tol_for

pytestmark = pytest.mark.gpu

PATHS = [rocs.PATH_AUTO, rocs.PATH_GENERAL]


@pytest.fixture(autouse=True)
def _reset_path():
    yield
    rocs.set_path(rocs.PATH_AUTO)
    rocs.last_device_status()


def _run(cfg, co, k, sample=None, path=rocs.PATH_AUTO):
    rocs.set_path(path)
    d = wl.glm_inputs(cfg, co)
    P = wl.fm_projection_weight(cfg, k)
    plan = rocs.plan_create(to_dev(co), co)
    outs = rocs.glm_fm_projection(plan, to_dev(d["XR"]), to_dev(d["XC"]), to_dev(P))
    F = ref.glm_fm_projection(co, d["XR"], d["XC"], P, sample=sample)
    if F.shape[0] == 0:
        return 0.0
    m = np.repeat(np.arange(cfg.R), np.diff(co))
    sel = (lambda a: a) if sample is None else (lambda a: a[sample])
    return max(rel_err(sel(to_host_f64(outs["FC"])), F[:, cfg.n_r:]),
               rel_err(sel(to_host_f64(outs["FR"])[m]), F[:, :cfg.n_r]))


def test_config1_fp32_every_element():
    cfg = wl.CONFIGS[1]
    assert _run(cfg, wl.cand_offsets(cfg), k=5) <= tol_for("f32")


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("k", [8, 16])
@pytest.mark.parametrize("d_emb", [64, 128, 192, 256])
def test_bf16_ragged_segments_and_tail_tile(path, k, d_emb):
    # empty requests, single candidates, segments that straddle the 8-candidate tiles, N % 8 != 0
    co = wl.offsets_from_counts([1, 0, 9, 8, 33, 7, 0, 133])
    cfg = wl.CONFIGS[4].with_(R=len(co) - 1, d_emb=d_emb)
    assert _run(cfg, co, k, path=path) <= tol_for("bf16")


@pytest.mark.parametrize("path", PATHS)
def test_bf16_shapes_outside_the_streaming_kernel(path):
    co = wl.offsets_from_counts([20, 3, 41])
    cfg = wl.CONFIGS[4].with_(R=3, n_r=24, n_c=8, d_emb=64)
    assert _run(cfg, co, 12, path=path) <= tol_for("bf16")
    cfg = wl.CONFIGS[4].with_(R=3, n_r=8, n_c=16, d_emb=32)
    assert _run(cfg, co, 16, path=path) <= tol_for("bf16")


def test_wide_request_group():
    co = wl.offsets_from_counts([3, 70, 5])
    cfg = wl.CONFIGS[4].with_(R=3, n_r=64, d_emb=256)
    assert _run(cfg, co, 16) <= tol_for("bf16")


def test_many_tiles_per_cta():
    # more tiles than CTAs: every CTA goes around its ring several times and changes request mid-run
    g = np.random.default_rng(7)
    co = wl.offsets_from_counts(g.integers(0, 200, size=120).tolist())
    cfg = wl.CONFIGS[4].with_(R=len(co) - 1)
    assert _run(cfg, co, 16) <= tol_for("bf16")


def test_config4_full_size_sampled():
    cfg = wl.CONFIGS[4]
    co = wl.cand_offsets(cfg)
    sample = wl.stratified_sample(co, n_uniform=512, n_small_requests=0, cfg_id=4)
    assert _run(cfg, co, 16, sample=sample) <= tol_for("bf16")


def _bits(t):
    return t.contiguous().view(torch.uint8).cpu().numpy().reshape(t.shape[0], -1)


@pytest.mark.parametrize("path", PATHS)
def test_candidate_isolation_is_bit_exact(path):
    rocs.set_path(path)
    co = wl.offsets_from_counts([130, 1, 64, 300, 5, 150])
    cfg = wl.CONFIGS[4].with_(R=6)
    d = wl.glm_inputs(cfg, co)
    P = to_dev(wl.fm_projection_weight(cfg, 16))
    plan = rocs.plan_create(to_dev(co), co)
    XR, XC = to_dev(d["XR"]), to_dev(d["XC"])
    N = int(co[-1])
    j = int(co[3]) + 77
    seg = slice(int(co[2]), int(co[3]))
    base = _bits(rocs.glm_fm_projection(plan, XR, XC, P)["FC"])
    assert np.array_equal(base, _bits(rocs.glm_fm_projection(plan, XR, XC, P)["FC"])), "not deterministic"
    XC2 = XC.clone()
    XC2[j] += 0.5
    pert = _bits(rocs.glm_fm_projection(plan, XR, XC2, P)["FC"])
    others = np.ones(N, bool)
    others[j] = False
    assert np.array_equal(base[others], pert[others]) and not np.array_equal(base[j], pert[j])
    XR2 = XR.clone()
    XR2[2] += 0.5
    pert = _bits(rocs.glm_fm_projection(plan, XR2, XC, P)["FC"])
    outside = np.ones(N, bool)
    outside[seg] = False
    assert np.array_equal(base[outside], pert[outside]), "a request leaked into another segment"
    assert np.all(np.any(base[seg] != pert[seg], axis=1))


def test_error_codes():
    co = wl.offsets_from_counts([4, 4])
    cfg = wl.CONFIGS[4].with_(R=2)
    d = wl.glm_inputs(cfg, co)
    plan = rocs.plan_create(to_dev(co), co)
    XR, XC, P = to_dev(d["XR"]), to_dev(d["XC"]), to_dev(wl.fm_projection_weight(cfg, 16))
    with pytest.raises(rocs.RocsError) as e:
        rocs.glm_fm_projection(plan, XR, XC, P, workspace=torch.empty(16, dtype=torch.uint8, device="cuda"))
    assert e.value.code == -5  # ROCS_ERR_WORKSPACE
    need = rocs.glm_fm_projection_workspace(plan, cfg.d_emb, 16)
    assert need >= 2 * 16 * cfg.d_emb * 4 and need % 256 == 0
