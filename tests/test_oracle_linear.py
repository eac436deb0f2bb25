"""Pins for the oracle's GLM linear (Eq. 4 two-group form, Eq. 14 of Section 4.1).

Nothing here retypes the oracle's loop: each test fixes the result through a library
routine on a case that reduces to it, a closed form, an invariant the paper states, or a
pure-Python brute force.
"""
import numpy as np
import pytest

from oracle import rocs_ref as ref
from paper_2607_27744_b200 import workloads as wl


def _tiny(dtype="f32", bias=True):
    cfg = wl.CONFIGS[1].with_(dtype=dtype)
    return cfg, wl.linear_inputs(cfg, bias=bias)


def test_special_case_one_candidate_per_request_is_a_plain_matmul():
    # R == N: the broadcast is the identity, so Eq. 4 is numpy.matmul on the concatenation.
    g = np.random.default_rng(1)
    R, d_req, d_cand, d_out = 7, 5, 3, 4
    XR, XC = g.standard_normal((R, d_req)), g.standard_normal((R, d_cand))
    W, b = g.standard_normal((d_out, d_req + d_cand)), g.standard_normal(d_out)
    co = np.arange(R + 1, dtype=np.int32)
    Y = ref.ikbo_linear(co, XR, XC, W, bias=b)
    np.testing.assert_allclose(Y, np.concatenate([XR, XC], 1) @ W.T + b, rtol=1e-13, atol=1e-13)


def test_special_case_no_request_features_is_a_plain_matmul():
    g = np.random.default_rng(2)
    XC, W = g.standard_normal((11, 6)), g.standard_normal((5, 6))
    co = np.array([0, 3, 3, 11], np.int32)
    Y = ref.ikbo_linear(co, None, XC, W)
    np.testing.assert_allclose(Y, XC @ W.T, rtol=1e-13, atol=1e-13)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_against_numpy_on_replicated_request_rows(dtype):
    # General case through a library: replicate x^R with numpy.repeat, then matmul.
    cfg, d = _tiny(dtype)
    co = d["cand_offsets"]
    XR, XC, W = (wl.to_f64(d[k]) for k in ("XR", "XC", "W"))
    U = np.concatenate([np.repeat(XR, np.diff(co), axis=0), XC], axis=1)
    want = np.maximum(U @ W.T + d["bias"].astype(np.float64), 0.0)
    got = ref.ikbo_linear(co, d["XR"], d["XC"], d["W"], bias=d["bias"], relu=True)
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-12)
    assert (got == 0).any() and (got > 0).any()  # the ReLU really clips something


def test_decomposed_form_equals_materialised_form():
    # Eq. 14: Z[m_i] + W_CC x^C_i  ==  [W_CR | W_CC] [x^R[m_i]; x^C_i]
    cfg, d = _tiny()
    co = d["cand_offsets"]
    Y = ref.ikbo_linear(co, d["XR"], d["XC"], d["W"], bias=d["bias"])
    Z, Yd = ref.ikbo_linear_decomposed(co, d["XR"], d["XC"], d["W"], bias=d["bias"])
    np.testing.assert_allclose(Yd, Y, rtol=1e-12, atol=1e-12)
    # Z is the request-only product: W_CR X^R + b
    want_Z = wl.to_f64(d["XR"]) @ wl.to_f64(d["W"])[:, :cfg.d_req].T + d["bias"]
    np.testing.assert_allclose(Z, want_Z, rtol=1e-12, atol=1e-12)


def test_closed_form_identity_block_copies_request_row():
    # W = [I | 0]: every candidate of request r gets x^R[r] exactly.
    R, d_req, d_cand = 3, 4, 2
    XR = np.arange(R * d_req, dtype=np.float64).reshape(R, d_req) + 1
    co = np.array([0, 2, 2, 5], np.int32)   # request 1 has no candidates
    XC = np.full((5, d_cand), 7.0)
    W = np.concatenate([np.eye(d_req), np.zeros((d_req, d_cand))], 1)
    Y = ref.ikbo_linear(co, XR, XC, W)
    assert np.array_equal(Y, XR[[0, 0, 2, 2, 2]])


def test_closed_form_one_hot_inputs_select_weight_columns():
    # x^R = e_a, x^C = e_b  ->  y = W[:, a] + W[:, d_req + b]
    g = np.random.default_rng(3)
    d_req, d_cand, d_out = 4, 3, 5
    W = g.standard_normal((d_out, d_req + d_cand))
    XR = np.eye(d_req)[[2, 0]]
    XC = np.eye(d_cand)[[1, 1, 2]]
    co = np.array([0, 1, 3], np.int32)
    Y = ref.ikbo_linear(co, XR, XC, W)
    want = np.stack([W[:, 2] + W[:, 4 + 1], W[:, 0] + W[:, 4 + 1], W[:, 0] + W[:, 4 + 2]])
    assert np.array_equal(Y, want)
    # a transposed weight, or swapped W_CR / W_CC blocks, cannot produce these columns


def test_zero_candidate_block_gives_shared_rows():
    # W_CC = 0 -> all candidates of a request get the same output (Eq. 11).
    cfg, d = _tiny()
    W = d["W"].copy()
    W[:, cfg.d_req:] = 0
    co = d["cand_offsets"]
    Y = ref.ikbo_linear(co, d["XR"], d["XC"], W)
    for r in range(cfg.R):
        seg = Y[co[r]:co[r + 1]]
        assert np.array_equal(seg, np.repeat(seg[:1], len(seg), 0))


def test_glm_invariant_candidate_isolation():
    # Eq. 1: perturbing candidate j changes only row j; perturbing request r changes
    # exactly the rows of segment r.
    cfg, d = _tiny()
    co = d["cand_offsets"]
    base = ref.ikbo_linear(co, d["XR"], d["XC"], d["W"])
    j = int(co[2])  # first candidate of request 2
    XC2 = d["XC"].copy()
    XC2[j] += 1.0
    out = ref.ikbo_linear(co, d["XR"], XC2, d["W"])
    changed = np.any(out != base, axis=1)
    assert changed[j] and changed.sum() == 1
    XR2 = d["XR"].copy()
    XR2[1] += 1.0
    out = ref.ikbo_linear(co, XR2, d["XC"], d["W"])
    changed = np.any(out != base, axis=1)
    want = np.zeros_like(changed)
    want[co[1]:co[2]] = True
    assert np.array_equal(changed, want)


def test_brute_force_python_loops():
    cfg = wl.CONFIGS[1].with_(R=3, d_req=5, d_cand=4, d_out=3)
    d = wl.linear_inputs(cfg, bias=True)
    co = d["cand_offsets"]
    XR, XC, W = d["XR"].tolist(), d["XC"].tolist(), d["W"].tolist()
    got = ref.ikbo_linear(co, d["XR"], d["XC"], d["W"], bias=d["bias"], relu=True)
    for r in range(cfg.R):
        for i in range(co[r], co[r + 1]):
            for o in range(cfg.d_out):
                acc = 0.0
                for k in range(cfg.d_req):
                    acc += W[o][k] * XR[r][k]
                for k in range(cfg.d_cand):
                    acc += W[o][cfg.d_req + k] * XC[i][k]
                acc += float(d["bias"][o])
                assert got[i, o] == pytest.approx(max(acc, 0.0), rel=1e-12, abs=1e-12)


def test_sampled_rows_match_full_run():
    cfg, d = _tiny()
    co = d["cand_offsets"]
    full = ref.ikbo_linear(co, d["XR"], d["XC"], d["W"])
    idx = np.array([int(co[-1]) - 1, 0, int(co[1])], np.int64)
    part = ref.ikbo_linear(co, d["XR"], d["XC"], d["W"], sample=idx)
    assert np.array_equal(part, full[idx])


def test_bf16_storage_is_widened_exactly():
    # 1.0078125 = 1 + 2^-7 is exactly representable in bf16; 3 * it must be exact in fp64.
    x = wl.f32_to_bf16_bits(np.array([[1.0078125]], np.float32))
    w = wl.f32_to_bf16_bits(np.array([[3.0]], np.float32))
    Y = ref.ikbo_linear(np.array([0, 1], np.int32), None, x, w)
    assert Y[0, 0] == 3.0234375


def test_amortised_flops_formula():
    # C_amort(N) = C_C + C_R / N (Section 5.1, Metrics) on config 2, layer 1.
    cfg = wl.CONFIGS[2]
    C_C = 2 * cfg.d_cand * cfg.d_out
    C_R = 2 * cfg.d_req * cfg.d_out
    assert C_C == 524288 and C_R == 1048576
    assert C_C + C_R / 512 == 526336
