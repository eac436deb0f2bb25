"""Every output element at full size: the IKBO kernels against the materialised-broadcast GPU path.

The fp64 oracle is slow by design, so the full-size parity tests compare a stratified sample with it.
Here the comparator is the dense path the paper starts from (request tensors replicated per
candidate, then torch library kernels), which covers EVERY row of the full-size outputs.  The
comparator is itself held against the oracle on a sample first, so agreement with it means
something.  Both sides store bf16, so the bound is the bf16 tolerance on
max |a - b| / max |b| per output tensor.
"""
import numpy as np
import pytest
import torch

import bench
from oracle import rocs_ref as ref
from paper_2607_27744_b200 import binding as rocs, workloads as wl
from _util import rel_err, to_dev, to_host_f64, tol_for

pytestmark = pytest.mark.gpu


def _rel(a, b):
    """max |a - b| / max |b| on the device, in fp32, chunked so no full-size fp32 copy is needed."""
    worst, top = 0.0, 0.0
    a2, b2 = a.reshape(a.shape[0], -1), b.reshape(b.shape[0], -1)
    for i in range(0, a2.shape[0], 1 << 16):
        x, y = a2[i:i + (1 << 16)].float(), b2[i:i + (1 << 16)].float()
        assert bool(torch.isfinite(x).all())
        worst = max(worst, float((x - y).abs().max()))
        top = max(top, float(y.abs().max()))
    return worst / top


def test_linear_config2_every_row():
    cfg = wl.CONFIGS[2]
    co = wl.cand_offsets(cfg)
    d = wl.linear_inputs(cfg, co)
    XR, XC, W = to_dev(d["XR"]), to_dev(d["XC"]), to_dev(d["W"])
    counts = to_dev(np.diff(co).astype(np.int64))
    dense = bench.materialised_linear(torch, XR, XC, W, counts, relu=True)
    sample = wl.stratified_sample(co, n_uniform=96, n_small_requests=0, cfg_id=2)
    want = ref.ikbo_linear(co, d["XR"], d["XC"], d["W"], relu=True, sample=sample)
    assert rel_err(to_host_f64(dense)[sample], want) <= tol_for("bf16")
    plan = rocs.plan_create(to_dev(co), co)
    y = rocs.ikbo_linear(plan, XR, XC, W[:, :cfg.d_req], W[:, cfg.d_req:], relu=True)
    assert _rel(y, dense) <= tol_for("bf16")


def test_linear_config5_every_row():
    # Zipf segments: a third of the 32-row slabs hold several requests
    cfg = wl.CONFIGS[5]
    co = wl.cand_offsets(cfg)
    d = wl.linear_inputs(cfg, co)
    XR, XC, W = to_dev(d["XR"]), to_dev(d["XC"]), to_dev(d["W"])
    plan = rocs.plan_create(to_dev(co), co)
    y = rocs.ikbo_linear(plan, XR, XC, W[:, :cfg.d_req], W[:, cfg.d_req:], relu=False)
    row2req = torch.repeat_interleave(torch.arange(cfg.R, device="cuda"), to_dev(np.diff(co).astype(np.int64)))
    N = int(co[-1])
    worst, top = 0.0, 0.0
    sample = wl.stratified_sample(co, n_uniform=64, n_small_requests=4, cfg_id=5)
    checked_against_oracle = False
    for a in range(0, N, 1 << 18):
        b = min(N, a + (1 << 18))
        dense = torch.cat([XR[row2req[a:b]], XC[a:b]], dim=1) @ W.t()
        if not checked_against_oracle:
            s = sample[sample < b - a]
            want = ref.ikbo_linear(co, d["XR"], d["XC"], d["W"], sample=s)
            assert rel_err(to_host_f64(dense)[s], want) <= tol_for("bf16")
            checked_against_oracle = True
        worst = max(worst, float((y[a:b].float() - dense.float()).abs().max()))
        top = max(top, float(dense.float().abs().max()))
    assert worst / top <= tol_for("bf16")


@pytest.mark.parametrize("dh", [64, 128, 32])
def test_attention_config3_every_row(dh):
    cfg = wl.CONFIGS[3] if dh == 64 else wl.CONFIGS[3].with_(H=8 * 64 // dh, dh=dh)
    co, so = wl.cand_offsets(cfg), wl.seq_offsets(cfg)
    d = wl.dca_inputs(cfg, co, so)
    Q, K, V = to_dev(d["Q"]), to_dev(d["K"]), to_dev(d["V"])
    dense = bench.materialised_dca(torch, Q, K, V, co, so, chunk_bytes=2 << 30)
    sample = wl.stratified_sample(co, n_uniform=48, n_small_requests=1, cfg_id=3)
    want = ref.dca_attention(co, so, d["Q"], d["K"], d["V"], sample=sample)
    assert rel_err(to_host_f64(dense)[sample], want) <= tol_for("bf16")
    plan = rocs.plan_create(to_dev(co), co)
    o = rocs.dca_attention(plan, Q, K, V, to_dev(so))
    assert _rel(o, dense) <= tol_for("bf16")
    assert rocs.last_device_status() == 0


def test_interaction_config4_every_row():
    cfg = wl.CONFIGS[4]
    co = wl.cand_offsets(cfg)
    d = wl.glm_inputs(cfg, co)
    XR, XC, W = to_dev(d["XR"]), to_dev(d["XC"]), to_dev(d["W"])
    counts = to_dev(np.diff(co).astype(np.int64))
    dense = bench.materialised_glm(torch, XR, XC, W, counts, cfg.n_r, cfg.n_ro)[:, cfg.n_ro:]   # candidate rows of O
    sample = wl.stratified_sample(co, n_uniform=64, n_small_requests=0, cfg_id=4)
    _, want = ref.glm_interaction(co, d["XR"], d["XC"], W=d["W"], n_ro=cfg.n_ro, n_co=cfg.n_co, sample=sample)
    assert rel_err(to_host_f64(dense)[sample], want[:, cfg.n_ro:]) <= tol_for("bf16")
    plan = rocs.plan_create(to_dev(co), co)
    out = rocs.glm_interaction(plan, XR, XC, W, cfg.n_ro, cfg.n_co, want_raw=False)
    assert _rel(out["OC"], dense) <= tol_for("bf16")
