"""Candidate isolation (Eq. 1) on the GPU at the sizes and launch geometry the benchmark times:
perturbing one candidate leaves the bits of every other candidate's output alone, perturbing one
request moves only its own segment, and nothing foreign (another request's rows behind the end of
a sequence, even Inf or NaN) reaches a request's output.  Comparisons run on the device."""
import numpy as np
import pytest
import torch

from paper_2607_27744_b200 import binding as rocs, workloads as wl
from _util import to_dev

pytestmark = pytest.mark.gpu


def _rows_differ(a, b):
    """bool [N]: which candidates' outputs differ in any bit."""
    n = a.shape[0]
    return (a.reshape(n, -1).view(torch.int16) != b.reshape(n, -1).view(torch.int16)).any(dim=1)


def _pick(co, rank):
    """A candidate in the middle of the rank-th largest request, and that request."""
    counts = np.diff(co)
    r = int(np.argsort(-counts)[rank])
    return r, int(co[r]) + int(counts[r]) // 2 + 7


def test_attention_isolation_config3_full_size():
    cfg = wl.CONFIGS[3]
    co, so = wl.cand_offsets(cfg), wl.seq_offsets(cfg)
    d = wl.dca_inputs(cfg, co, so)
    Q, K, V, sod = to_dev(d["Q"]), to_dev(d["K"]), to_dev(d["V"]), to_dev(so)
    plan = rocs.plan_create(to_dev(co), co)
    base = rocs.dca_attention(plan, Q, K, V, sod)
    again = rocs.dca_attention(plan, Q, K, V, sod)
    assert not _rows_differ(base, again).any(), "not run-to-run deterministic"
    for rank in (0, 20, 63):                      # a large, a middling and the smallest request
        r, j = _pick(co, rank)
        j = min(j, int(co[r + 1]) - 1)
        Q2 = Q.clone()
        Q2[j] *= 1.5
        diff = _rows_differ(base, rocs.dca_attention(plan, Q2, K, V, sod))
        assert bool(diff[j]) and int(diff.sum()) == 1, "another candidate's output changed"
        K2, V2 = K.clone(), V.clone()
        K2[int(so[r]):int(so[r + 1])] *= 0.5
        V2[int(so[r]):int(so[r + 1])] += 1.0
        diff = _rows_differ(base, rocs.dca_attention(plan, Q, K2, V2, sod))
        inside = torch.zeros_like(diff)
        inside[int(co[r]):int(co[r + 1])] = True
        assert not (diff & ~inside).any(), "a request leaked into another segment"
        assert bool(diff[inside].all())
    rocs.last_device_status()


def test_attention_ignores_foreign_rows_behind_the_end_of_a_sequence():
    """The last key block of a request reaches into the next request's K/V rows (or past the end of
    the tensor).  Whatever sits there -- huge values, Inf, NaN -- must not change the request's output."""
    cfg = wl.CONFIGS[5].with_(R=5)
    co = wl.offsets_from_counts([130, 40, 300, 1, 77])
    so = wl.offsets_from_counts([150, 20, 300, 128, 33])     # ragged: every tail block is partial
    d = wl.dca_inputs(cfg, co, so)
    Q, K, V, sod = to_dev(d["Q"]), to_dev(d["K"]), to_dev(d["V"]), to_dev(so)
    plan = rocs.plan_create(to_dev(co), co)
    base = rocs.dca_attention(plan, Q, K, V, sod)
    assert torch.isfinite(base.float()).all()
    for r in (1, 2, 4):                            # poison the first rows of request r
        for poison in (float("nan"), float("inf"), -3e38):
            K2, V2 = K.clone(), V.clone()
            V2[int(so[r]):int(so[r]) + 8] = poison
            K2[int(so[r]) + 1:int(so[r]) + 4] = poison
            out = rocs.dca_attention(plan, Q, K2, V2, sod)
            outside = torch.ones(int(co[-1]), dtype=torch.bool, device="cuda")
            outside[int(co[r]):int(co[r + 1])] = False
            assert not (_rows_differ(base, out) & outside).any(), "foreign rows reached another request's output"
            assert torch.isfinite(out[outside].float()).all()
    rocs.last_device_status()


def test_interaction_isolation_config4_full_size():
    cfg = wl.CONFIGS[4]
    co = wl.cand_offsets(cfg)
    g = wl.glm_inputs(cfg, co)
    XR, XC, W = to_dev(g["XR"]), to_dev(g["XC"]), to_dev(g["W"])
    plan = rocs.plan_create(to_dev(co), co)
    run = lambda xr, xc: rocs.glm_interaction(plan, xr, xc, W, cfg.n_ro, cfg.n_co)
    base, again = run(XR, XC), run(XR, XC)
    for k in ("YC", "OC", "YR", "OR"):
        assert torch.equal(base[k].view(torch.int16), again[k].view(torch.int16)), "not run-to-run deterministic"
    r = 77
    j = int(co[r]) + 500
    XC2 = XC.clone()
    XC2[j] += 0.5
    pert = run(XR, XC2)
    for k in ("YC", "OC"):
        diff = _rows_differ(base[k], pert[k])
        assert bool(diff[j]) and int(diff.sum()) == 1, f"{k}: another candidate's output changed"
    for k in ("YR", "OR"):
        assert torch.equal(base[k].view(torch.int16), pert[k].view(torch.int16)), "request rows depend on a candidate"
    XR2 = XR.clone()
    XR2[r] += 0.5
    pert = run(XR2, XC)
    inside = torch.zeros(int(co[-1]), dtype=torch.bool, device="cuda")
    inside[int(co[r]):int(co[r + 1])] = True
    for k in ("YC", "OC"):
        diff = _rows_differ(base[k], pert[k])
        assert not (diff & ~inside).any(), f"{k}: a request leaked into another segment"
        assert bool(diff[inside].all())
    for k in ("YR", "OR"):
        diff = _rows_differ(base[k], pert[k])
        assert bool(diff[r]) and int(diff.sum()) == 1
    rocs.last_device_status()


def test_projected_fm_isolation_config4_full_size():
    cfg = wl.CONFIGS[4]
    co = wl.cand_offsets(cfg)
    g = wl.glm_inputs(cfg, co)
    XR, XC, P = to_dev(g["XR"]), to_dev(g["XC"]), to_dev(wl.fm_projection_weight(cfg, 16))
    plan = rocs.plan_create(to_dev(co), co)
    run = lambda xr, xc: rocs.glm_fm_projection(plan, xr, xc, P)
    base, again = run(XR, XC), run(XR, XC)
    for k in ("FC", "FR"):
        assert torch.equal(base[k].view(torch.int16), again[k].view(torch.int16)), "not run-to-run deterministic"
    r = 5
    j = int(co[r]) + 1023
    XC2 = XC.clone()
    XC2[j] += 0.5
    pert = run(XR, XC2)
    diff = _rows_differ(base["FC"], pert["FC"])
    assert bool(diff[j]) and int(diff.sum()) == 1, "another candidate's output changed"
    assert torch.equal(base["FR"].view(torch.int16), pert["FR"].view(torch.int16))
    XR2 = XR.clone()
    XR2[r] += 0.5
    pert = run(XR2, XC)
    inside = torch.zeros(int(co[-1]), dtype=torch.bool, device="cuda")
    inside[int(co[r]):int(co[r + 1])] = True
    diff = _rows_differ(base["FC"], pert["FC"])
    assert not (diff & ~inside).any(), "a request leaked into another segment"
    assert bool(diff[inside].all())
    rocs.last_device_status()
