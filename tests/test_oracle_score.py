"""Pins for the oracle's proxy score (window softmax, group/window sum, max-pool).

The attention weights are the scaled-dot-product softmax of Eq. 1 (Sec. 3.1); the
observation-window reading is the conventional SnapKV one.  None of these checks calls the
oracle to produce its own expected value: they use the row-sum identity, closed forms,
library routines (torch.softmax, scipy max filter, torch max_pool1d) and limits.
"""
import numpy as np
import pytest
import torch
from scipy.ndimage import maximum_filter1d


def _rand(rng, *shape):
    return rng.standard_normal(shape).astype(np.float32)


def test_softmax_rows_sum_to_one_and_are_causal(oracle):
    rng = np.random.default_rng(0)
    G, w, d, T = 3, 5, 16, 77
    q, k = _rand(rng, G, w, d), _rand(rng, T, d)
    p = oracle.window_softmax(q, k)
    assert p.shape == (G * w, T)
    np.testing.assert_allclose(p.sum(axis=1), 1.0, rtol=0, atol=1e-13)
    n = T - w
    for g in range(G):
        for i in range(w):
            row = p[g * w + i]
            assert np.all(row[n + i + 1:] == 0.0)          # future keys masked
            assert np.all(row[:n + i + 1] > 0.0)           # every visible key has mass


def test_mass_conservation(oracle):
    rng = np.random.default_rng(1)
    G, w, d, T = 2, 4, 8, 50
    q, k = _rand(rng, G, w, d), _rand(rng, T, d)
    raw, _ = oracle.score_head(q, k, kp=1)
    assert raw.shape == (T,)
    np.testing.assert_allclose(raw.sum(), G * w, rtol=1e-13)


def test_identical_keys_closed_form(oracle):
    # all keys equal => every visible key gets 1/(n+i+1) in row i => raw_j = G * sum_i 1/(n+i+1)
    rng = np.random.default_rng(2)
    G, w, d, T = 3, 6, 16, 40
    q = _rand(rng, G, w, d)
    k = np.tile(_rand(rng, 1, d), (T, 1))
    raw, pooled = oracle.score_head(q, k, kp=7)
    n = T - w
    expect = G * sum(1.0 / (n + i + 1) for i in range(w))
    np.testing.assert_allclose(raw[:n], expect, rtol=1e-13)
    np.testing.assert_allclose(pooled, np.float32(expect), rtol=1e-6)
    # window column n+t is visible to rows i >= t only
    for t in range(w):
        np.testing.assert_allclose(raw[n + t], G * sum(1.0 / (n + i + 1) for i in range(t, w)), rtol=1e-13)


def test_zero_queries_give_uniform_attention(oracle):
    G, w, d, T = 2, 3, 8, 20
    q = np.zeros((G, w, d), np.float32)
    k = _rand(np.random.default_rng(3), T, d)
    raw, _ = oracle.score_head(q, k, kp=1)
    n = T - w
    np.testing.assert_allclose(raw[:n], G * sum(1.0 / (n + i + 1) for i in range(w)), rtol=1e-13)


def test_single_row_is_a_library_softmax(oracle):
    # w=1, G=1: the raw score vector is one softmax row over all T keys with scale 1/sqrt(d)
    rng = np.random.default_rng(4)
    d, T = 32, 300
    q, k = _rand(rng, 1, 1, d), _rand(rng, T, d)
    raw, _ = oracle.score_head(q, k, kp=1)
    logits = torch.from_numpy(k).double() @ torch.from_numpy(q[0, 0]).double() / np.sqrt(d)
    ref = torch.softmax(logits, dim=0).numpy()
    np.testing.assert_allclose(raw, ref, rtol=1e-12, atol=0)


def test_explicit_scale_overrides_default(oracle):
    rng = np.random.default_rng(5)
    d, T = 16, 64
    q, k = _rand(rng, 1, 1, d), _rand(rng, T, d)
    raw, _ = oracle.score_head(q, k, kp=1, scale=0.37)
    logits = torch.from_numpy(k).double() @ torch.from_numpy(q[0, 0]).double() * np.float64(np.float32(0.37))
    np.testing.assert_allclose(raw, torch.softmax(logits, 0).numpy(), rtol=1e-12)


def test_dominant_key_takes_all_mass(oracle):
    rng = np.random.default_rng(6)
    G, w, d, T = 2, 4, 8, 60
    q = np.abs(_rand(rng, G, w, d)) + 0.5
    k = 0.01 * _rand(rng, T, d)
    k[17] = 50.0                      # logit >> all others for every (positive) query
    raw, _ = oracle.score_head(q, k, kp=1)
    assert abs(raw[17] - G * w) < 1e-9
    assert raw[:T - w].sum() - raw[17] < 1e-9


def test_shift_invariance(oracle):
    # adding a vector orthogonal to every query... simpler: adding c*q-independent constant to all
    # logits of a row leaves softmax unchanged; realise it by appending a channel: q_c = 1, k_c = const
    rng = np.random.default_rng(7)
    G, w, d, T = 2, 3, 8, 40
    q, k = _rand(rng, G, w, d), _rand(rng, T, d)
    raw0, _ = oracle.score_head(q, k, kp=1, scale=0.25)
    q1 = np.concatenate([q, np.ones((G, w, 1), np.float32)], axis=2)
    k1 = np.concatenate([k, np.full((T, 1), 3.0, np.float32)], axis=1)
    raw1, _ = oracle.score_head(q1, k1, kp=1, scale=0.25)
    np.testing.assert_allclose(raw1, raw0, rtol=1e-12)


def test_dense_attention_with_library_ops(oracle):
    # the same quantity written with dense torch ops (masked softmax), float64
    rng = np.random.default_rng(8)
    G, w, d, T = 4, 8, 32, 200
    n = T - w
    q, k = _rand(rng, G, w, d), _rand(rng, T, d)
    raw, pooled = oracle.score_head(q, k, kp=5)
    Q = torch.from_numpy(q).double().reshape(G * w, d)
    K = torch.from_numpy(k).double()
    logits = Q @ K.T / np.sqrt(d)
    pos = torch.arange(T)[None, :]
    qpos = (n + torch.arange(w)).repeat(G)[:, None]
    logits = logits.masked_fill(pos > qpos, float("-inf"))
    ref = torch.softmax(logits, dim=1).sum(dim=0)
    np.testing.assert_allclose(raw, ref.numpy(), rtol=1e-11)
    ref_pool = torch.nn.functional.max_pool1d(ref[None, None, :n], 5, stride=1, padding=2)[0, 0]
    np.testing.assert_array_equal(pooled, ref_pool.numpy().astype(np.float32))


def test_bf16_inputs_are_widened_exactly(oracle):
    rng = np.random.default_rng(9)
    G, w, d, T = 2, 4, 16, 64
    qb = torch.from_numpy(_rand(rng, G, w, d)).bfloat16()
    kb = torch.from_numpy(_rand(rng, T, d)).bfloat16()
    raw_b, pooled_b = oracle.score_head(qb.view(torch.int16).numpy().view(np.uint16),
                                        kb.view(torch.int16).numpy().view(np.uint16), kp=3)
    raw_f, pooled_f = oracle.score_head(qb.float().numpy(), kb.float().numpy(), kp=3)
    np.testing.assert_array_equal(raw_b, raw_f)
    np.testing.assert_array_equal(pooled_b, pooled_f)


@pytest.mark.parametrize("kp", [1, 3, 5, 7, 9])
def test_max_pool_against_library_filter(oracle, kp):
    rng = np.random.default_rng(10 + kp)
    for n in (1, 2, 5, 33, 200):
        raw = rng.random(n)
        got = oracle.max_pool(raw, kp)
        ref = maximum_filter1d(raw, size=kp, mode="constant", cval=-np.inf)
        np.testing.assert_array_equal(got, ref)
        assert np.all(got >= raw)
        if kp == 1:
            np.testing.assert_array_equal(got, raw)


def test_pool_does_not_see_window_columns(oracle):
    # a huge raw score in the first window column must not leak into pooled[n-1]
    rng = np.random.default_rng(20)
    G, w, d, T = 1, 4, 8, 30
    n = T - w
    q = np.abs(_rand(rng, G, w, d)) + 0.5
    k = 0.01 * _rand(rng, T, d)
    k[n] = 50.0
    raw, pooled = oracle.score_head(q, k, kp=7)
    assert raw[n] > 3.9
    assert pooled.max() < 1.0


def test_score_all_heads_layout(oracle):
    # q [S][L][H*G][w][d]: query heads h*G..h*G+G-1 belong to KV head h
    rng = np.random.default_rng(21)
    S, L, H, G, w, d, T = 2, 2, 3, 2, 3, 8, 24
    q = _rand(rng, S, L, H * G, w, d)
    k = _rand(rng, S, L, H, T, d)
    sc = oracle.score(q, k, G, kp=3)
    assert sc.shape == (S, L * H, T - w)
    for s in range(S):
        for l in range(L):
            for h in range(H):
                _, pooled = oracle.score_head(q[s, l, h * G:(h + 1) * G], k[s, l, h], kp=3)
                np.testing.assert_array_equal(sc[s, l * H + h], pooled)


def test_tiny_values_flush_to_zero(oracle):
    # probabilities below the smallest normal float are stored as +0
    G, w, d, T = 1, 1, 2, 8
    q = np.array([[[40.0, 0.0]]], np.float32)
    k = np.zeros((T, d), np.float32)
    k[:, 0] = -10.0
    k[T - 1, 0] = 10.0                         # window key: logit gap 800/sqrt(2) >> 88
    _, pooled = oracle.score_head(q, k, kp=1)
    assert np.all(pooled == 0.0) and not np.any(np.signbit(pooled))
