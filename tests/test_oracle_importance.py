"""Pins of the oracle's oracle-importance function (Sec. 4.1, Eq. "oracle_importance"; App. E).

I_j = max over decode steps k of (attention weight of step k on cached position j) x || v_j W_O ||_2,
summed over the query heads of a KV head before the maximum, each layer normalised to unit mass.
Pinned by what the definition fixes: a library softmax times a library vector norm for one step and an
identity projection; closed forms (identical keys, zero queries); monotonicity in K_max; a decode key
that absorbs a step's attention; grouped heads that double the score; scaling by the projection;
the normalisation's unit mass; and the window positions being left out.
"""
import numpy as np
import pytest
import torch

from oracle import lukv_oracle as O


def _rand(S, L, H, G, d, T, Kmax, Dm, seed):
    rng = np.random.default_rng(seed)
    q = rng.standard_normal((S, L, H * G, Kmax, d)).astype(np.float32)
    k = rng.standard_normal((S, L, H, T, d)).astype(np.float32)
    v = rng.standard_normal((S, L, H, T, d)).astype(np.float32)
    kd = rng.standard_normal((S, L, H, Kmax, d)).astype(np.float32)
    wo = (rng.standard_normal((L, H * G, d, Dm)) / np.sqrt(d)).astype(np.float32)
    return q, k, v, kd, wo


def test_one_step_identity_projection_is_library_softmax_times_library_norm():
    S, L, H, G, d, T, w = 1, 1, 2, 1, 16, 50, 5
    q, k, v, _, _ = _rand(S, L, H, G, d, T, 1, d, 0)
    eye = np.broadcast_to(np.eye(d, dtype=np.float32), (L, H, d, d)).copy()
    got = O.importance(q, k, v, eye, G, w, normalize=False)
    for h in range(H):
        logits = torch.from_numpy(k[0, 0, h].astype(np.float64)) @ torch.from_numpy(q[0, 0, h, 0].astype(np.float64))
        a = torch.softmax(logits / np.sqrt(d), dim=0)
        want = (a * torch.linalg.vector_norm(torch.from_numpy(v[0, 0, h].astype(np.float64)), dim=1))[: T - w]
        np.testing.assert_allclose(got[0, h], want.numpy(), rtol=1e-6)


def test_identical_keys_and_zero_queries_give_uniform_attention():
    S, L, H, G, d, T, w, Kmax, Dm = 1, 1, 1, 2, 8, 40, 4, 3, 12
    q, k, v, kd, wo = _rand(S, L, H, G, d, T, Kmax, Dm, 1)
    k[:] = k[0, 0, 0, 0]                      # every cached key the same: weights 1/T whatever the query
    got = O.importance(q, k, v, wo, G, w, normalize=False)
    norms = [np.linalg.norm(v[0, 0, 0].astype(np.float64) @ wo[0, g].astype(np.float64), axis=1) for g in range(G)]
    np.testing.assert_allclose(got[0, 0], (sum(norms) / T)[: T - w], rtol=1e-6)
    # zero queries with decode keys: step k spreads its weight over T + k keys, so the first step is the maximum
    q0 = np.zeros_like(q)
    rng = np.random.default_rng(2)
    k2 = rng.standard_normal(k.shape).astype(np.float32)
    got = O.importance(q0, k2, v, wo, G, w, k_dec=kd, normalize=False)
    np.testing.assert_allclose(got[0, 0], (sum(norms) / (T + 1))[: T - w], rtol=1e-6)


def test_monotone_in_the_number_of_decode_steps():
    S, L, H, G, d, T, w, Dm = 1, 2, 2, 2, 8, 60, 6, 10
    q, k, v, kd, wo = _rand(S, L, H, G, d, T, 5, Dm, 3)
    prev = None
    for Kmax in range(1, 6):
        cur = O.importance(q[:, :, :, :Kmax], k, v, wo, G, w, k_dec=kd[:, :, :, :Kmax], normalize=False)
        if prev is not None:
            assert np.all(cur >= prev)          # a maximum over more steps
        prev = cur
    assert np.any(cur > O.importance(q[:, :, :, :1], k, v, wo, G, w, k_dec=kd[:, :, :, :1], normalize=False))


def test_a_dominant_decode_key_takes_the_attention_of_its_step():
    S, L, H, G, d, T, w, Dm = 1, 1, 1, 1, 8, 30, 3, 8
    q, k, v, kd, wo = _rand(S, L, H, G, d, T, 2, Dm, 4)
    kd[0, 0, 0, 1] = 100.0 * q[0, 0, 0, 1]     # step 2's own key absorbs step 2's attention
    both = O.importance(q, k, v, wo, G, w, k_dec=kd, normalize=False)
    first = O.importance(q[:, :, :, :1], k, v, wo, G, w, k_dec=kd[:, :, :, :1], normalize=False)
    np.testing.assert_allclose(both, first, rtol=1e-6)   # step 2 contributes nothing to any cached position


def test_grouped_query_heads_add_and_the_projection_scales():
    S, L, H, d, T, w, Kmax, Dm = 1, 1, 2, 8, 33, 4, 3, 6
    q, k, v, kd, wo = _rand(S, L, H, 1, d, T, Kmax, Dm, 5)
    one = O.importance(q, k, v, wo, 1, w, k_dec=kd, normalize=False)
    q2 = np.repeat(q, 2, axis=2)                # two identical query heads per KV head ...
    wo2 = np.repeat(wo, 2, axis=1)              # ... with the same projection slice
    two = O.importance(q2, k, v, wo2, 2, w, k_dec=kd, normalize=False)
    np.testing.assert_allclose(two, 2.0 * one, rtol=1e-6)
    np.testing.assert_allclose(O.importance(q, k, v, 3.0 * wo, 1, w, k_dec=kd, normalize=False), 3.0 * one, rtol=1e-6)
    # a projection that annihilates the values leaves no importance
    assert np.all(O.importance(q, k, v, 0.0 * wo, 1, w, k_dec=kd, normalize=False) == 0.0)


def test_normalisation_gives_every_layer_unit_mass_and_keeps_ratios():
    S, L, H, G, d, T, w, Kmax, Dm = 2, 3, 2, 2, 8, 40, 5, 3, 7
    q, k, v, kd, wo = _rand(S, L, H, G, d, T, Kmax, Dm, 6)
    wo[1] *= 50.0                               # one layer with much larger projected values
    raw = O.importance(q, k, v, wo, G, w, k_dec=kd, normalize=False).astype(np.float64)
    nrm = O.importance(q, k, v, wo, G, w, k_dec=kd, normalize=True).astype(np.float64)
    n = T - w
    for s in range(S):
        for l in range(L):
            blk = slice(l * H, (l + 1) * H)
            assert abs(nrm[s, blk].sum() - 1.0) < 1e-5
            np.testing.assert_allclose(nrm[s, blk], raw[s, blk] / raw[s, blk].sum(), rtol=2e-6)
    assert nrm.shape == (S, L * H, n)


def test_window_positions_are_left_out_and_bf16_inputs_widen_exactly():
    S, L, H, G, d, T, Kmax, Dm = 1, 1, 1, 2, 8, 24, 2, 8
    q, k, v, kd, wo = _rand(S, L, H, G, d, T, Kmax, Dm, 7)
    full = O.importance(q, k, v, wo, G, 1, k_dec=kd, normalize=False)
    cut = O.importance(q, k, v, wo, G, 7, k_dec=kd, normalize=False)
    np.testing.assert_array_equal(cut[0, 0], full[0, 0, : T - 7])

    def to_bf16_bits(a):
        return (torch.from_numpy(a).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16))

    def widen(a):
        return torch.from_numpy(a).to(torch.bfloat16).float().numpy()

    got = O.importance(to_bf16_bits(q), to_bf16_bits(k), to_bf16_bits(v), to_bf16_bits(wo), G, 3, k_dec=to_bf16_bits(kd))
    want = O.importance(widen(q), widen(k), widen(v), widen(wo), G, 3, k_dec=widen(kd))
    np.testing.assert_array_equal(got, want)
