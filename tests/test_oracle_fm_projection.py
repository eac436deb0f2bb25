"""Pins for the oracle's projected factorization machine: F = G P, G the masked interaction of Eq. 9-10."""
import numpy as np
import pytest

from oracle import rocs_ref as ref
from paper_2607_27744_b200 import workloads as wl


def _tiny(dtype="f32", k=5):
    cfg = wl.CONFIGS[1].with_(dtype=dtype)
    d = wl.glm_inputs(cfg)
    P = wl.fm_projection_weight(cfg, k)
    return cfg, d, P


def test_identity_projection_reduces_to_the_interaction_operator():
    # P = I (k = n): F is the masked interaction matrix itself, which has its own pins
    cfg, d, _ = _tiny()
    n = cfg.n_r + cfg.n_c
    P = np.eye(n, dtype=np.float32)
    F = ref.glm_fm_projection(d["cand_offsets"], d["XR"], d["XC"], P)
    G, _ = ref.glm_interaction(d["cand_offsets"], d["XR"], d["XC"])
    assert np.array_equal(F, G)


def test_column_selection_and_linearity_in_P():
    cfg, d, P = _tiny()
    co = d["cand_offsets"]
    n = cfg.n_r + cfg.n_c
    G, _ = ref.glm_interaction(co, d["XR"], d["XC"])
    # a one-hot column of P picks one column of G: catches a transposed P or a transposed G
    for b in (0, cfg.n_r - 1, cfg.n_r, n - 1):
        E = np.zeros((n, 2), np.float32)
        E[b, 1] = 1.0
        F = ref.glm_fm_projection(co, d["XR"], d["XC"], E)
        assert np.all(F[:, :, 0] == 0)
        assert np.array_equal(F[:, :, 1], G[:, :, b])
    Pf = wl.to_f64(P)
    F1 = ref.glm_fm_projection(co, wl.to_f64(d["XR"]), wl.to_f64(d["XC"]), Pf)
    F2 = ref.glm_fm_projection(co, wl.to_f64(d["XR"]), wl.to_f64(d["XC"]), 2.0 * Pf)
    assert np.array_equal(F2, 2.0 * F1)


def test_closed_forms():
    # every embedding equal to c * ones(d): G = c^2 d everywhere below the mask
    n_r, n_c, dd, k, c = 3, 2, 8, 4, 0.5
    XR = np.full((1, n_r, dd), c)
    XC = np.full((1, n_c, dd), c)
    g = np.random.default_rng(3)
    P = g.standard_normal((n_r + n_c, k))
    F = ref.glm_fm_projection(np.array([0, 1], np.int32), XR, XC, P)
    np.testing.assert_allclose(F[0, :n_r], np.tile(c * c * dd * P[:n_r].sum(0), (n_r, 1)), rtol=1e-13)
    np.testing.assert_allclose(F[0, n_r:], np.tile(c * c * dd * P.sum(0), (n_c, 1)), rtol=1e-13)
    # orthonormal rows: G = I, so F = P
    E = np.eye(dd)
    F = ref.glm_fm_projection(np.array([0, 1], np.int32), E[None, :n_r], E[None, n_r:n_r + n_c], P)
    assert np.array_equal(F[0], P)
    # zero candidate embeddings: the candidate rows vanish, the request rows do not
    F = ref.glm_fm_projection(np.array([0, 1], np.int32), g.standard_normal((1, n_r, dd)), np.zeros((1, n_c, dd)), P)
    assert np.all(F[0, n_r:] == 0) and np.any(F[0, :n_r] != 0)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_against_numpy_on_the_materialised_matrix(dtype):
    cfg, d, P = _tiny(dtype)
    co = d["cand_offsets"]
    XR, XC, Pf = wl.to_f64(d["XR"]), wl.to_f64(d["XC"]), wl.to_f64(P)
    F = ref.glm_fm_projection(co, d["XR"], d["XC"], P)
    n_r = cfg.n_r
    for r in range(cfg.R):
        for i in range(co[r], co[r + 1]):
            X = np.concatenate([XR[r], XC[i]], 0)
            G = X @ X.T
            G[:n_r, n_r:] = 0.0
            np.testing.assert_allclose(F[i], G @ Pf, rtol=1e-12, atol=1e-12)


def test_request_rows_never_see_candidates_and_ignore_P_C():
    cfg, d, P = _tiny()
    co = d["cand_offsets"]
    n_r = cfg.n_r
    F = ref.glm_fm_projection(co, d["XR"], d["XC"], P)
    XC2 = (d["XC"] * 3.0 + 1.0).astype(d["XC"].dtype)
    P2 = P.copy()
    P2[n_r:] += 1.0
    F2 = ref.glm_fm_projection(co, d["XR"], XC2, P2)
    assert np.array_equal(F[:, :n_r], F2[:, :n_r])        # Eq. 1: request side is candidate-invariant
    assert not np.array_equal(F[:, n_r:], F2[:, n_r:])
    for r in range(cfg.R):                                 # and the same for every candidate of a request
        for i in range(co[r], co[r + 1]):
            assert np.array_equal(F[i, :n_r], F[co[r], :n_r])


def test_isolation():
    cfg, d, P = _tiny()
    co = d["cand_offsets"]
    F = ref.glm_fm_projection(co, d["XR"], d["XC"], P)
    i = int(co[1])  # first candidate of request 1
    XC2 = d["XC"].copy()
    XC2[i] = XC2[i] * -2.0 + 0.5
    F2 = ref.glm_fm_projection(co, d["XR"], XC2, P)
    changed = np.any(F != F2, axis=(1, 2))
    assert changed[i] and changed.sum() == 1


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_request_once_form_equals_materialised_form(dtype):
    cfg, d, P = _tiny(dtype)
    co = d["cand_offsets"]
    F = ref.glm_fm_projection(co, d["XR"], d["XC"], P)
    FR, FC = ref.glm_fm_projection_decomposed(co, d["XR"], d["XC"], P)
    n_r = cfg.n_r
    scale = np.abs(F).max()
    np.testing.assert_allclose(FC, F[:, n_r:], rtol=0, atol=1e-12 * scale)
    for r in range(cfg.R):
        if co[r + 1] > co[r]:
            np.testing.assert_allclose(FR[r], F[co[r], :n_r], rtol=0, atol=1e-12 * scale)


def test_brute_force_python_loops():
    g = np.random.default_rng(5)
    n_r, n_c, dd, k = 2, 3, 4, 2
    co = np.array([0, 2, 2, 3], np.int32)
    XR = g.standard_normal((3, n_r, dd))
    XC = g.standard_normal((3, n_c, dd))
    P = g.standard_normal((n_r + n_c, k))
    F = ref.glm_fm_projection(co, XR, XC, P)
    m = [0, 0, 2]
    for i in range(3):
        rows = [XR[m[i], a] for a in range(n_r)] + [XC[i, a] for a in range(n_c)]
        for a in range(n_r + n_c):
            for c in range(k):
                acc = 0.0
                for b in range(n_r + n_c):
                    if a < n_r and b >= n_r:
                        continue  # lower-triangular block mask of Eq. 9
                    dot = sum(rows[a][e] * rows[b][e] for e in range(dd))
                    acc += dot * P[b, c]
                assert abs(F[i, a, c] - acc) < 1e-12


def test_sampled_rows_match_full_run():
    cfg, d, P = _tiny()
    co = d["cand_offsets"]
    F = ref.glm_fm_projection(co, d["XR"], d["XC"], P)
    sample = np.array([int(co[-1]) - 1, 0, 3], np.int64)
    Fs = ref.glm_fm_projection(co, d["XR"], d["XC"], P, sample=sample)
    assert np.array_equal(Fs, F[sample])
