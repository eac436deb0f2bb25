"""Group-local normalisation (Eq. 7) folded into the layers around it: the split layer leaves each
row's sums, the next layer applies scale and shift to its accumulators, the normalised rows are never
written.  Checked against the oracle's composition  linear( group_norm( ReLU(split layer) ) )."""
import numpy as np
import pytest
import torch

from oracle import rocs_ref as ref
from paper_2607_27744_b200 import binding as rocs, workloads as wl
from _util import rel_err, to_dev, to_host_f64, tol_for

pytestmark = pytest.mark.gpu


def _case(counts, d_req, d_cand, d_mid, d_out, seed):
    cfg = wl.CONFIGS[2].with_(R=len(counts), d_req=d_req, d_cand=d_cand, d_out=d_mid)
    co = wl.offsets_from_counts(counts)
    lin = wl.linear_inputs(cfg, co, bias=True)
    g = np.random.default_rng(seed)
    W2 = wl.store((g.standard_normal((d_out, d_mid)) / np.sqrt(d_mid)).astype(np.float32), "bf16")
    gamma = (1.0 + 0.2 * g.standard_normal(d_mid)).astype(np.float64)
    beta = (0.3 * g.standard_normal(d_mid)).astype(np.float64)
    b2 = g.standard_normal(d_out).astype(np.float32)
    return cfg, co, lin, W2, gamma, beta, b2


@pytest.mark.parametrize("kind", [rocs.NORM_LAYER, rocs.NORM_RMS])
@pytest.mark.parametrize("counts,dims", [([700, 3, 41, 0, 1300, 17, 300], (256, 128, 192, 256)),
                                          ([2048, 2048], (512, 256, 1024, 512))])
def test_norm_folded_into_the_next_layer_matches_the_oracle_composition(kind, counts, dims):
    d_req, d_cand, d_mid, d_out = dims
    cfg, co, lin, W2, gamma, beta, b2 = _case(counts, d_req, d_cand, d_mid, d_out, seed=11)
    eps = 1e-5
    # oracle: split layer (ReLU) -> group norm with gain / offset -> plain layer
    h = ref.ikbo_linear(co, lin["XR"], lin["XC"], lin["W"], bias=lin["bias"], relu=True)
    n = ref.group_norm(h, gamma, beta if kind == rocs.NORM_LAYER else None, eps,
                       ref.LAYER_NORM if kind == rocs.NORM_LAYER else ref.RMS_NORM)
    want = ref.ikbo_linear(wl.offsets_from_counts([n.shape[0]]), None, n, wl.to_f64(W2), bias=b2.astype(np.float64))
    # GPU: gain folded into the weight columns, offset into the bias (host-side preparation, fp64 then bf16)
    W2f = wl.to_f64(W2)
    W2g = wl.store((W2f * gamma[None, :]).astype(np.float32), "bf16")
    b2f = (b2.astype(np.float64) + (W2f @ beta if kind == rocs.NORM_LAYER else 0.0)).astype(np.float32)
    W = to_dev(lin["W"])
    plan = rocs.plan_create(to_dev(co), co)
    Y, stats = rocs.ikbo_linear_stats(plan, to_dev(lin["XR"]), to_dev(lin["XC"]), W[:, :d_req], W[:, d_req:],
                                      bias=to_dev(lin["bias"]), relu=True)
    # the sums themselves
    hs = to_host_f64(Y)
    got_stats = to_host_f64(stats)
    assert rel_err(got_stats[:, 0], hs.sum(1)) <= 1e-2 and rel_err(got_stats[:, 1], (hs * hs).sum(1)) <= 1e-2
    W2g_d = to_dev(W2g)
    wbar = rocs.weight_row_sums(W2g_d)
    assert rel_err(to_host_f64(wbar), wl.to_f64(W2g).sum(1)) <= 1e-5
    out = rocs.linear_normed(Y, stats, W2g_d, wbar if kind == rocs.NORM_LAYER else None, to_dev(b2f), eps, kind)
    assert rel_err(to_host_f64(out), want) <= tol_for("bf16")
    # and against the unfused GPU pipeline (stand-alone normalisation kernel, then the plain layer)
    g_d = torch.from_numpy(gamma.astype(np.float32)).to(torch.bfloat16).cuda()
    b_d = torch.from_numpy(beta.astype(np.float32)).to(torch.bfloat16).cuda() if kind == rocs.NORM_LAYER else None
    unfused = rocs.linear(rocs.group_norm(Y, g_d, b_d, eps, kind), to_dev(W2), to_dev(b2))
    assert rel_err(to_host_f64(out), to_host_f64(unfused)) <= 2 * tol_for("bf16")
    rocs.last_device_status()


def test_small_batches_take_the_stored_output_for_the_sums_and_the_fold_is_refused():
    cfg, co, lin, W2, gamma, beta, b2 = _case([5, 40, 1], 64, 32, 64, 256, seed=3)
    W = to_dev(lin["W"])
    plan = rocs.plan_create(to_dev(co), co)
    Y, stats = rocs.ikbo_linear_stats(plan, to_dev(lin["XR"]), to_dev(lin["XC"]), W[:, :64], W[:, 64:], relu=True)
    hs = to_host_f64(Y)
    assert rel_err(to_host_f64(stats)[:, 0], hs.sum(1)) <= 1e-5
    assert rel_err(to_host_f64(stats)[:, 1], (hs * hs).sum(1)) <= 1e-5
    with pytest.raises(rocs.RocsError) as e:           # 46 rows: not a shape of the wide-layer kernel
        rocs.linear_normed(Y, stats, to_dev(W2), None, None, 1e-5, rocs.NORM_RMS)
    assert e.value.code == -3
