"""Pins for the oracle's group-local normalisation (Eq. 7)."""
import numpy as np
import pytest
import torch

from oracle import rocs_ref as ref
from paper_2607_27744_b200 import workloads as wl


def _x(M=7, d=24, seed=1):
    g = np.random.default_rng(seed)
    return g.standard_normal((M, d)) * 3.0 + 0.7, g.standard_normal(d), g.standard_normal(d)


def test_layer_norm_against_the_library_routine():
    X, gamma, beta = _x()
    want = torch.nn.functional.layer_norm(torch.from_numpy(X), (X.shape[1],), torch.from_numpy(gamma),
                                          torch.from_numpy(beta), eps=1e-5).numpy()
    np.testing.assert_allclose(ref.group_norm(X, gamma, beta, 1e-5, ref.LAYER_NORM), want, rtol=1e-12, atol=1e-12)
    want = torch.nn.functional.layer_norm(torch.from_numpy(X), (X.shape[1],), eps=1e-3).numpy()
    np.testing.assert_allclose(ref.group_norm(X, None, None, 1e-3, ref.LAYER_NORM), want, rtol=1e-12, atol=1e-12)


def test_rms_norm_against_the_library_routine():
    X, gamma, _ = _x()
    want = torch.nn.functional.rms_norm(torch.from_numpy(X), (X.shape[1],), torch.from_numpy(gamma), eps=1e-6).numpy()
    np.testing.assert_allclose(ref.group_norm(X, gamma, None, 1e-6, ref.RMS_NORM), want, rtol=1e-12, atol=1e-12)


def test_closed_forms_and_invariances():
    X, gamma, beta = _x()
    d = X.shape[1]
    # statistics of the normalised row
    Y = ref.group_norm(X, None, None, 0.0, ref.LAYER_NORM)
    np.testing.assert_allclose(Y.mean(1), 0.0, atol=1e-13)
    np.testing.assert_allclose((Y ** 2).mean(1), 1.0, rtol=1e-12)
    Y = ref.group_norm(X, None, None, 0.0, ref.RMS_NORM)
    np.testing.assert_allclose((Y ** 2).mean(1), 1.0, rtol=1e-12)
    # LayerNorm ignores a shift and a positive scale of its input, RMSNorm only the scale
    np.testing.assert_allclose(ref.group_norm(5.0 * X + 2.0, gamma, beta, 0.0, ref.LAYER_NORM),
                               ref.group_norm(X, gamma, beta, 0.0, ref.LAYER_NORM), rtol=1e-11, atol=1e-11)
    np.testing.assert_allclose(ref.group_norm(5.0 * X, gamma, None, 0.0, ref.RMS_NORM),
                               ref.group_norm(X, gamma, None, 0.0, ref.RMS_NORM), rtol=1e-12)
    assert not np.allclose(ref.group_norm(X + 2.0, gamma, None, 0.0, ref.RMS_NORM),
                           ref.group_norm(X, gamma, None, 0.0, ref.RMS_NORM))
    # a two-valued row: +-1 after LayerNorm; a constant row: 0 (LayerNorm with eps) and sign * gamma (RMSNorm)
    row = np.array([[2.0, 6.0] * (d // 2)])
    assert np.allclose(ref.group_norm(row, None, None, 0.0, ref.LAYER_NORM), np.array([[-1.0, 1.0] * (d // 2)]))
    const = np.full((1, d), -4.0)
    assert np.all(ref.group_norm(const, gamma, beta, 1e-5, ref.LAYER_NORM) == beta)
    np.testing.assert_allclose(ref.group_norm(const, gamma, None, 0.0, ref.RMS_NORM), -gamma[None], rtol=1e-14)
    # eps enters under the square root, once
    one = np.array([[3.0, -3.0]])
    np.testing.assert_allclose(ref.group_norm(one, None, None, 7.0, ref.RMS_NORM), one / 4.0, rtol=1e-14)
    np.testing.assert_allclose(ref.group_norm(one, None, None, 7.0, ref.LAYER_NORM), one / 4.0, rtol=1e-14)


def test_rows_are_independent_and_bf16_input_is_widened_exactly():
    X, gamma, beta = _x(M=5)
    Y = ref.group_norm(X, gamma, beta)
    X2 = X.copy()
    X2[2] = -X2[2] + 1.0
    Y2 = ref.group_norm(X2, gamma, beta)
    assert np.array_equal(np.delete(Y, 2, 0), np.delete(Y2, 2, 0)) and not np.array_equal(Y[2], Y2[2])
    Xb = wl.store(X.astype(np.float32), "bf16")
    gb = wl.store(gamma.astype(np.float32), "bf16")
    np.testing.assert_allclose(ref.group_norm(Xb, gb, None, 1e-5, ref.RMS_NORM),
                               ref.group_norm(wl.to_f64(Xb), wl.to_f64(gb), None, 1e-5, ref.RMS_NORM), rtol=0, atol=0)


def test_statistics_over_concatenated_groups_would_break_the_invariant():
    # Eq. 7's point: group-local statistics leave the request side untouched by the candidate;
    # statistics over [x^R ; x^C] do not
    g = np.random.default_rng(4)
    xr, xc1, xc2 = g.standard_normal((1, 16)), g.standard_normal((1, 8)), 4.0 * g.standard_normal((1, 8))
    local1, local2 = ref.group_norm(xr), ref.group_norm(xr)
    assert np.array_equal(local1, local2)
    joint1 = ref.group_norm(np.concatenate([xr, xc1], 1))[:, :16]
    joint2 = ref.group_norm(np.concatenate([xr, xc2], 1))[:, :16]
    assert not np.allclose(joint1, joint2)


def test_brute_force_python_loops():
    X, gamma, beta = _x(M=3, d=5)
    for kind in (ref.LAYER_NORM, ref.RMS_NORM):
        Y = ref.group_norm(X, gamma, beta, 1e-2, kind)
        for i in range(3):
            mean = sum(X[i]) / 5
            if kind == ref.LAYER_NORM:
                var = sum((v - mean) ** 2 for v in X[i]) / 5
                want = [(X[i, e] - mean) / (var + 1e-2) ** 0.5 * gamma[e] + beta[e] for e in range(5)]
            else:
                ms = sum(v * v for v in X[i]) / 5
                want = [X[i, e] / (ms + 1e-2) ** 0.5 * gamma[e] for e in range(5)]
            assert max(abs(a - b) for a, b in zip(Y[i], want)) < 1e-13
