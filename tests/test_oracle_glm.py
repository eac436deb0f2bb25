"""Pins for the oracle's GLM factorization machine (Eq. 9-10) and row-axis compression (Eq. 5-6)."""
import numpy as np
import pytest

from oracle import rocs_ref as ref
from paper_2607_27744_b200 import workloads as wl


def _tiny(dtype="f32"):
    cfg = wl.CONFIGS[1].with_(dtype=dtype, n_ro=3, n_co=2)
    return cfg, wl.glm_inputs(cfg)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_against_numpy_gram_matrix_with_block_mask(dtype):
    cfg, d = _tiny(dtype)
    co = d["cand_offsets"]
    XR, XC, W = wl.to_f64(d["XR"]), wl.to_f64(d["XC"]), wl.to_f64(d["W"])
    G, O = ref.glm_interaction(co, d["XR"], d["XC"], d["W"], cfg.n_ro, cfg.n_co)
    n_r = cfg.n_r
    Wm = W.copy()
    Wm[: cfg.n_ro, n_r:] = 0.0
    for r in range(cfg.R):
        for i in range(co[r], co[r + 1]):
            X = np.concatenate([XR[r], XC[i]], 0)
            want = X @ X.T
            want[:n_r, n_r:] = 0.0
            np.testing.assert_allclose(G[i], want, rtol=1e-12, atol=1e-12)
            np.testing.assert_allclose(O[i], Wm @ want, rtol=1e-12, atol=1e-12)


def test_closed_forms():
    # orthonormal rows -> G is the identity with its upper-right block (already 0) masked
    n_r, n_c, d = 3, 2, 8
    E = np.eye(d)
    XR, XC = E[None, :n_r], E[None, n_r:n_r + n_c]
    G, _ = ref.glm_interaction(np.array([0, 1], np.int32), XR, XC)
    assert np.array_equal(G[0], np.eye(n_r + n_c))
    # candidate rows equal to request rows -> CR block equals the RR block; upper right stays 0
    g = np.random.default_rng(11)
    XR = g.standard_normal((1, 3, 6))
    G, _ = ref.glm_interaction(np.array([0, 1], np.int32), XR, XR.copy())
    assert np.array_equal(G[0, 3:, :3], G[0, :3, :3])
    assert np.all(G[0, :3, 3:] == 0) and np.any(G[0, 3:, 3:] != 0)
    # CC block symmetric, diagonal = squared norms
    XC = g.standard_normal((1, 4, 6))
    G, _ = ref.glm_interaction(np.array([0, 1], np.int32), XR, XC)
    CC = G[0, 3:, 3:]
    np.testing.assert_allclose(CC, CC.T, rtol=1e-14)
    np.testing.assert_allclose(np.diag(CC), (XC[0] ** 2).sum(1), rtol=1e-13)
    # CR block is X^C X^R^T and not its transpose
    np.testing.assert_allclose(G[0, 3:, :3], XC[0] @ XR[0].T, rtol=1e-13, atol=1e-14)


def test_mask_is_inside_the_operator_request_rows_never_see_candidates():
    cfg, d = _tiny()
    co = d["cand_offsets"]
    G, O = ref.glm_interaction(co, d["XR"], d["XC"], d["W"], cfg.n_ro, cfg.n_co)
    XC2 = (d["XC"] * 3.0 + 1.0).astype(d["XC"].dtype)
    G2, O2 = ref.glm_interaction(co, d["XR"], XC2, d["W"], cfg.n_ro, cfg.n_co)
    assert np.array_equal(G[:, :cfg.n_r], G2[:, :cfg.n_r])       # Y^R
    assert np.array_equal(O[:, :cfg.n_ro], O2[:, :cfg.n_ro])     # O^R
    assert not np.array_equal(O[:, cfg.n_ro:], O2[:, cfg.n_ro:])
    # sharing identity (Eq. 11): request-side outputs identical across a request's candidates
    for r in range(cfg.R):
        seg = G[co[r]:co[r + 1], :cfg.n_r]
        assert np.array_equal(seg, np.repeat(seg[:1], len(seg), 0))


def test_decomposed_form_equals_materialised_form():
    cfg, d = _tiny()
    co = d["cand_offsets"]
    G, O = ref.glm_interaction(co, d["XR"], d["XC"], d["W"], cfg.n_ro, cfg.n_co)
    YR, YC, OR, OC = ref.glm_interaction_decomposed(co, d["XR"], d["XC"], d["W"], cfg.n_ro, cfg.n_co)
    m = np.repeat(np.arange(cfg.R), np.diff(co))
    np.testing.assert_allclose(G[:, :cfg.n_r], YR[m], rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(G[:, cfg.n_r:], YC, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(O[:, :cfg.n_ro], OR[m], rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(O[:, cfg.n_ro:], OC, rtol=1e-12, atol=1e-12)


def test_identity_compression_reproduces_interaction():
    cfg = wl.CONFIGS[1]
    d = wl.glm_inputs(cfg)
    n = cfg.n_r + cfg.n_c
    G, O = ref.glm_interaction(d["cand_offsets"], d["XR"], d["XC"], np.eye(n, dtype=np.float32), cfg.n_r, cfg.n_c)
    assert np.array_equal(G, O)


def test_masked_weight_block_is_ignored():
    # W[0:n_ro, n_r:] must not matter (it is multiplied by the mask of Eq. 3).
    cfg, d = _tiny()
    W2 = d["W"].copy()
    W2[: cfg.n_ro, cfg.n_r:] += 5.0
    a = ref.glm_interaction(d["cand_offsets"], d["XR"], d["XC"], d["W"], cfg.n_ro, cfg.n_co)[1]
    b = ref.glm_interaction(d["cand_offsets"], d["XR"], d["XC"], W2, cfg.n_ro, cfg.n_co)[1]
    assert np.array_equal(a, b)


def test_isolation():
    cfg, d = _tiny()
    co = d["cand_offsets"]
    base = ref.glm_interaction(co, d["XR"], d["XC"], d["W"], cfg.n_ro, cfg.n_co)[1]
    XC2 = d["XC"].copy()
    j = int(co[3]) - 1
    XC2[j] += 1.0
    out = ref.glm_interaction(co, d["XR"], XC2, d["W"], cfg.n_ro, cfg.n_co)[1]
    changed = np.any(out != base, axis=(1, 2))
    assert changed[j] and changed.sum() == 1
    XR2 = d["XR"].copy()
    XR2[0] += 1.0
    out = ref.glm_interaction(co, XR2, d["XC"], d["W"], cfg.n_ro, cfg.n_co)[1]
    changed = np.any(out != base, axis=(1, 2))
    want = np.zeros_like(changed)
    want[co[0]:co[1]] = True
    assert np.array_equal(changed, want)


def test_brute_force_python_loops():
    cfg = wl.CONFIGS[1].with_(R=2, n_r=2, n_c=3, d_emb=4, n_ro=1, n_co=2)
    d = wl.glm_inputs(cfg)
    co = d["cand_offsets"]
    XR, XC, W = d["XR"].tolist(), d["XC"].tolist(), d["W"].tolist()
    G, O = ref.glm_interaction(co, d["XR"], d["XC"], d["W"], cfg.n_ro, cfg.n_co)
    n = 5
    for r in range(2):
        for i in range(co[r], co[r + 1]):
            X = XR[r] + XC[i]
            g = [[sum(X[a][e] * X[b][e] for e in range(4)) for b in range(n)] for a in range(n)]
            for a in range(2):
                for b in range(2, n):
                    g[a][b] = 0.0
            for a in range(n):
                for b in range(n):
                    assert G[i, a, b] == pytest.approx(g[a][b], rel=1e-12, abs=1e-13)
            for o in range(3):
                for b in range(n):
                    acc = sum((0.0 if (o < 1 and a >= 2) else W[o][a]) * g[a][b] for a in range(n))
                    assert O[i, o, b] == pytest.approx(acc, rel=1e-12, abs=1e-13)


def test_sampled_rows_match_full_run():
    cfg, d = _tiny()
    full = ref.glm_interaction(d["cand_offsets"], d["XR"], d["XC"], d["W"], cfg.n_ro, cfg.n_co)
    idx = np.array([2, 0], np.int64)
    part = ref.glm_interaction(d["cand_offsets"], d["XR"], d["XC"], d["W"], cfg.n_ro, cfg.n_co, sample=idx)
    assert np.array_equal(part[0], full[0][idx]) and np.array_equal(part[1], full[1][idx])
