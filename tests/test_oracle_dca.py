"""Pins for the oracle's group-wise cross attention, candidate side (Eq. 13)."""
import math

import numpy as np
import pytest
import torch

from oracle import rocs_ref as ref
from paper_2607_27744_b200 import workloads as wl


def _tiny(dtype="f32"):
    cfg = wl.CONFIGS[1].with_(dtype=dtype)
    return cfg, wl.dca_inputs(cfg)


def _softmax_attention(q, k, v, scale):
    """Textbook softmax(q k^T * scale) v for one head; q [m, dh], k, v [L, dh]."""
    s = (q @ k.T) * scale
    s = s - s.max(axis=1, keepdims=True)
    p = np.exp(s)
    return (p / p.sum(axis=1, keepdims=True)) @ v


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_against_textbook_numpy_attention_per_request(dtype):
    cfg, d = _tiny(dtype)
    co, so = d["cand_offsets"], d["seq_offsets"]
    Q, K, V = (wl.to_f64(d[k]) for k in "QKV")
    got = ref.dca_attention(co, so, d["Q"], d["K"], d["V"])
    scale = 1.0 / math.sqrt(cfg.dh)
    for r in range(cfg.R):
        for h in range(cfg.H):
            q = Q[co[r]:co[r + 1], 0, h]
            want = _softmax_attention(q, K[so[r]:so[r + 1], h], V[so[r]:so[r + 1], h], scale)
            np.testing.assert_allclose(got[co[r]:co[r + 1], 0, h], want, rtol=1e-11, atol=1e-12)


def test_against_torch_sdpa_independent_witness():
    # One request, several query tokens per candidate, explicit scale.
    g = np.random.default_rng(5)
    n, n_q, H, dh, L = 3, 4, 2, 8, 9
    Q, K, V = g.standard_normal((n, n_q, H, dh)), g.standard_normal((L, H, dh)), g.standard_normal((L, H, dh))
    co, so = np.array([0, n], np.int32), np.array([0, L], np.int32)
    got = ref.dca_attention(co, so, Q, K, V, scale=0.37)
    tq = torch.from_numpy(Q).permute(0, 2, 1, 3)                      # [n, H, n_q, dh]
    tk = torch.from_numpy(K).permute(1, 0, 2).unsqueeze(0).expand(n, -1, -1, -1)
    tv = torch.from_numpy(V).permute(1, 0, 2).unsqueeze(0).expand(n, -1, -1, -1)
    want = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, scale=0.37)
    np.testing.assert_allclose(got, want.permute(0, 2, 1, 3).numpy(), rtol=1e-10, atol=1e-12)


def test_default_scale_is_inverse_sqrt_dh():
    cfg, d = _tiny()
    a = ref.dca_attention(d["cand_offsets"], d["seq_offsets"], d["Q"], d["K"], d["V"])
    b = ref.dca_attention(d["cand_offsets"], d["seq_offsets"], d["Q"], d["K"], d["V"], scale=cfg.dh ** -0.5)
    c = ref.dca_attention(d["cand_offsets"], d["seq_offsets"], d["Q"], d["K"], d["V"], scale=1.0)
    assert np.allclose(a, b, rtol=1e-12, atol=1e-13) and not np.allclose(a, c, rtol=1e-3)


def test_shared_form_equals_materialised_form():
    # (S_{m_i}) W = (S W)_{m_i}: attending over copies or over the shared K/V is the same.
    cfg, d = _tiny()
    args = (d["cand_offsets"], d["seq_offsets"], d["Q"], d["K"], d["V"])
    np.testing.assert_allclose(ref.dca_attention_shared(*args), ref.dca_attention(*args), rtol=1e-13, atol=1e-14)


def test_closed_forms():
    g = np.random.default_rng(6)
    H, dh = 2, 4
    co = np.array([0, 2, 3, 5], np.int32)
    so = np.array([0, 5, 6, 9], np.int32)     # request 1 has a single key
    K, V = g.standard_normal((9, H, dh)), g.standard_normal((9, H, dh))
    # zero queries -> uniform weights -> mean of the request's V rows
    O = ref.dca_attention(co, so, np.zeros((5, 1, H, dh)), K, V)
    for r in range(3):
        for i in range(co[r], co[r + 1]):
            np.testing.assert_allclose(O[i, 0], V[so[r]:so[r + 1]].mean(0), rtol=1e-13, atol=1e-14)
    # a single key -> its value row, whatever the query
    Q = g.standard_normal((5, 1, H, dh))
    O = ref.dca_attention(co, so, Q, K, V)
    np.testing.assert_allclose(O[2, 0], V[5], rtol=1e-14, atol=1e-15)
    # identical keys -> mean of values
    K2 = K.copy()
    K2[0:5] = K[0]
    O2 = ref.dca_attention(co, so, Q, K2, V)
    np.testing.assert_allclose(O2[0, 0], V[0:5].mean(0), rtol=1e-12, atol=1e-13)
    # outputs lie in the per-dimension range of the request's values (convex combination)
    for r in range(3):
        seg = V[so[r]:so[r + 1]]
        for i in range(co[r], co[r + 1]):
            assert np.all(O[i, 0] <= seg.max(0) + 1e-12) and np.all(O[i, 0] >= seg.min(0) - 1e-12)


def test_peaked_query_selects_one_value_row():
    # orthogonal keys; a query that is a large multiple of key j returns V[j]; heads separate.
    dh, L = 8, 8
    K = np.zeros((L, 2, dh))
    K[:, 0] = np.eye(L)
    K[:, 1] = np.eye(L)[::-1]
    V = np.random.default_rng(7).standard_normal((L, 2, dh))
    Q = np.zeros((1, 1, 2, dh))
    Q[0, 0, 0] = 200.0 * np.eye(L)[3]
    Q[0, 0, 1] = 200.0 * np.eye(L)[3]           # head 1's key 4 is e_3
    O = ref.dca_attention(np.array([0, 1], np.int32), np.array([0, L], np.int32), Q, K, V, scale=1.0)
    np.testing.assert_allclose(O[0, 0, 0], V[3, 0], atol=1e-12)
    np.testing.assert_allclose(O[0, 0, 1], V[4, 1], atol=1e-12)


def test_large_scores_do_not_overflow():
    Q = np.full((1, 1, 1, 4), 400.0)
    K = np.stack([np.full((1, 4), 1.0), np.full((1, 4), 0.99)])
    V = np.array([[[1.0, 0, 0, 0]], [[0, 1.0, 0, 0]]])
    O = ref.dca_attention(np.array([0, 1], np.int32), np.array([0, 2], np.int32), Q, K, V, scale=1.0)
    assert np.all(np.isfinite(O))
    w = 1.0 / (1.0 + math.exp(-16.0))          # score gap 400*4*0.01 = 16
    np.testing.assert_allclose(O[0, 0, 0, :2], [w, 1 - w], rtol=1e-9)


def test_key_permutation_invariance():
    cfg, d = _tiny()
    co, so = d["cand_offsets"], d["seq_offsets"]
    base = ref.dca_attention(co, so, d["Q"], d["K"], d["V"])
    K, V = d["K"].copy(), d["V"].copy()
    perm = np.random.default_rng(8).permutation(int(so[1]))
    K[: so[1]] = K[: so[1]][perm]
    V[: so[1]] = V[: so[1]][perm]
    np.testing.assert_allclose(ref.dca_attention(co, so, d["Q"], K, V), base, rtol=1e-12, atol=1e-13)


def test_isolation_and_request_scope():
    cfg, d = _tiny()
    co, so = d["cand_offsets"], d["seq_offsets"]
    base = ref.dca_attention(co, so, d["Q"], d["K"], d["V"])
    Q2 = d["Q"].copy()
    j = int(co[1])
    Q2[j] *= 2.0
    changed = np.any(ref.dca_attention(co, so, Q2, d["K"], d["V"]) != base, axis=(1, 2, 3))
    assert changed[j] and changed.sum() == 1
    K2 = d["K"].copy()
    K2[so[2]: so[3]] += 0.5               # request 2's keys
    changed = np.any(ref.dca_attention(co, so, d["Q"], K2, d["V"]) != base, axis=(1, 2, 3))
    want = np.zeros_like(changed)
    want[co[2]: co[3]] = True
    assert np.array_equal(changed, want)


def test_empty_sequence_gives_zeros_and_ragged_lengths_work():
    g = np.random.default_rng(9)
    co = np.array([0, 2, 4], np.int32)
    so = np.array([0, 0, 3], np.int32)
    Q, K, V = g.standard_normal((4, 2, 1, 4)), g.standard_normal((3, 1, 4)), g.standard_normal((3, 1, 4))
    O = ref.dca_attention(co, so, Q, K, V)
    assert np.all(O[:2] == 0)
    want = _softmax_attention(Q[2:, :, 0].reshape(4, 4), K[:, 0], V[:, 0], 0.5).reshape(2, 2, 4)
    np.testing.assert_allclose(O[2:, :, 0], want, rtol=1e-12, atol=1e-13)


def test_brute_force_python_loops():
    cfg = wl.CONFIGS[1].with_(R=2, L_const=5, H=2, dh=3, n_q=2)
    d = wl.dca_inputs(cfg)
    co, so = d["cand_offsets"], d["seq_offsets"]
    Q, K, V = d["Q"].tolist(), d["K"].tolist(), d["V"].tolist()
    got = ref.dca_attention(co, so, d["Q"], d["K"], d["V"])
    scale = 1.0 / math.sqrt(3)
    for r in range(2):
        for i in range(co[r], co[r + 1]):
            for t in range(2):
                for h in range(2):
                    s = [scale * sum(Q[i][t][h][e] * K[j][h][e] for e in range(3)) for j in range(so[r], so[r + 1])]
                    mx = max(s)
                    p = [math.exp(x - mx) for x in s]
                    z = sum(p)
                    for e in range(3):
                        o = sum(p[jj] / z * V[so[r] + jj][h][e] for jj in range(len(p)))
                        assert got[i, t, h, e] == pytest.approx(o, rel=1e-12, abs=1e-13)


def test_sampled_rows_match_full_run():
    cfg, d = _tiny()
    full = ref.dca_attention(d["cand_offsets"], d["seq_offsets"], d["Q"], d["K"], d["V"])
    idx = np.array([3, 0, int(d["cand_offsets"][-1]) - 1], np.int64)
    part = ref.dca_attention(d["cand_offsets"], d["seq_offsets"], d["Q"], d["K"], d["V"], sample=idx)
    assert np.array_equal(part, full[idx])
