"""Pins for the oracle's top-b selection, gather and the whole path.

Selection is the top-b prefix of the positions ranked by the proxy (Sec. 3.2, M^pi(k);
Sec. 4.3 "Eviction") with ties going to the lower index; it is checked against a full
library sort.  Uniform budgets must reduce the whole path to per-head SnapKV, which is
written here with dense torch library ops, independently of the oracle.
"""
import numpy as np
import pytest
import torch


def test_select_matches_full_sort(oracle):
    rng = np.random.default_rng(0)
    for n, b in ((1, 0), (1, 1), (10, 3), (257, 100), (1000, 999), (1000, 1000)):
        sc = rng.random(n).astype(np.float32)
        kept = oracle.select(sc, b)
        order = np.argsort(-sc.astype(np.float64), kind="stable")
        np.testing.assert_array_equal(kept, np.sort(order[:b]))
        assert len(kept) == b and np.all(np.diff(kept) > 0)
        if 0 < b < n:
            evicted = np.setdiff1d(np.arange(n), kept)
            assert sc[kept].min() >= sc[evicted].max()


def test_select_ties_go_to_lower_index(oracle):
    sc = np.array([1, 5, 5, 5, 2, 5, 5, 0], np.float32)
    np.testing.assert_array_equal(oracle.select(sc, 3), [1, 2, 3])
    np.testing.assert_array_equal(oracle.select(sc, 4), [1, 2, 3, 5])
    np.testing.assert_array_equal(oracle.select(sc, 6), [1, 2, 3, 4, 5, 6])
    np.testing.assert_array_equal(oracle.select(np.zeros(9, np.float32), 4), [0, 1, 2, 3])
    # plateaus as produced by max-pooling
    rng = np.random.default_rng(1)
    sc = np.repeat(rng.random(50).astype(np.float32), 7)
    for b in (1, 10, 33, 200):
        kept = oracle.select(sc, b)
        order = np.lexsort((np.arange(len(sc)), -sc.astype(np.float64)))
        np.testing.assert_array_equal(kept, np.sort(order[:b]))


def test_select_values_match_library_topk(oracle):
    rng = np.random.default_rng(2)
    sc = rng.random(5000).astype(np.float32)
    b = 1234
    kept = oracle.select(sc, b)
    ref_vals = torch.topk(torch.from_numpy(sc), b).values.numpy()
    np.testing.assert_array_equal(np.sort(sc[kept]), np.sort(ref_vals))


def test_gather_layout_and_bytes(oracle):
    rng = np.random.default_rng(3)
    U, T, w, d = 5, 40, 4, 8
    n = T - w
    k = rng.standard_normal((U, T, d)).astype(np.float32)
    v = rng.standard_normal((U, T, d)).astype(np.float32)
    scores = rng.random((U, n)).astype(np.float32)
    budgets = np.array([0, 7, n, 1, 20], np.int32)
    offsets = np.concatenate([[0], np.cumsum(budgets + w)]).astype(np.int32)
    k_out, v_out, kept = oracle.select_gather(scores, budgets, offsets, k, v, w)
    assert k_out.shape == (budgets.sum() + U * w, d)
    for u in range(U):
        o, b = offsets[u], budgets[u]
        np.testing.assert_array_equal(kept[o:o + b], oracle.select(scores[u], int(b)))
        np.testing.assert_array_equal(kept[o + b:o + b + w], np.arange(n, T))
        for t in range(b + w):
            assert k_out[o + t].tobytes() == k[u, kept[o + t]].tobytes()
            assert v_out[o + t].tobytes() == v[u, kept[o + t]].tobytes()


def test_gather_bf16_rows_are_copied_bit_exactly(oracle):
    rng = np.random.default_rng(4)
    U, T, w, d = 2, 16, 2, 8
    k = rng.integers(0, 65536, (U, T, d)).astype(np.uint16)      # arbitrary bit patterns, NaNs included
    v = rng.integers(0, 65536, (U, T, d)).astype(np.uint16)
    scores = rng.random((U, T - w)).astype(np.float32)
    budgets = np.array([3, 5], np.int32)
    offsets = np.concatenate([[0], np.cumsum(budgets + w)]).astype(np.int32)
    k_out, v_out, kept = oracle.select_gather(scores, budgets, offsets, k, v, w)
    for u in range(U):
        for t in range(budgets[u] + w):
            r = offsets[u] + t
            np.testing.assert_array_equal(k_out[r], k[u, kept[r]])
            np.testing.assert_array_equal(v_out[r], v[u, kept[r]])


def _snapkv_with_library_ops(q, k, G, kp, b):
    """Per-head SnapKV with dense torch ops: q [H*G][w][d], k [H][T][d] -> kept score multisets."""
    HG, w, d = q.shape
    H, T, _ = k.shape
    n = T - w
    out = []
    for h in range(H):
        Q = torch.from_numpy(q[h * G:(h + 1) * G]).double().reshape(G * w, d)
        K = torch.from_numpy(k[h]).double()
        logits = Q @ K.T / np.sqrt(d)
        qpos = (n + torch.arange(w)).repeat(G)[:, None]
        logits = logits.masked_fill(torch.arange(T)[None, :] > qpos, float("-inf"))
        votes = torch.softmax(logits, dim=1)[:, :n].sum(dim=0)
        pooled = torch.nn.functional.max_pool1d(votes[None, None], kp, stride=1, padding=kp // 2)[0, 0]
        out.append(pooled.float())
    return out


def test_uniform_allocation_reduces_to_per_head_snapkv(oracle):
    rng = np.random.default_rng(5)
    S, L, H, G, w, d, T, kp, P = 1, 2, 2, 2, 4, 16, 64, 5, 9
    N, n, s = L * H, T - w, T // (P - 1)
    q = rng.standard_normal((S, L, H * G, w, d)).astype(np.float32)
    k = rng.standard_normal((S, L, H, T, d)).astype(np.float32)
    v = rng.standard_normal((S, L, H, T, d)).astype(np.float32)
    curves = np.zeros((N, P), np.float32)
    curves[:, 1:] = np.cumsum(np.arange(P - 1, 0, -1, dtype=np.float64))[None, :]   # identical, strictly concave
    b_each = 3 * s
    out = oracle.compress(q, k, v, curves, [N * b_each], G, kp)
    assert np.all(out["budgets"] == b_each)
    for l in range(L):
        pooled = _snapkv_with_library_ops(q[0, l], k[0, l], G, kp, b_each)
        for h in range(H):
            u = l * H + h
            o = out["offsets"][u]
            kept = out["kept_idx"][o:o + b_each]
            ref = pooled[h]
            np.testing.assert_allclose(out["scores"][0, u], ref.numpy(), rtol=1e-6)
            top_vals = torch.topk(ref, b_each).values.numpy()
            np.testing.assert_array_equal(np.sort(ref.numpy()[kept]), np.sort(top_vals))
            np.testing.assert_array_equal(out["kept_idx"][o + b_each:o + b_each + w], np.arange(n, T))
            np.testing.assert_array_equal(out["k_out"][o:o + b_each], k[0, l, h][kept])
            np.testing.assert_array_equal(out["v_out"][o:o + b_each], v[0, l, h][kept])


def test_compress_batch_is_per_sequence(oracle):
    rng = np.random.default_rng(6)
    S, L, H, G, w, d, T, kp, P = 2, 1, 3, 1, 2, 8, 32, 3, 5
    N, n = L * H, T - w
    q = rng.standard_normal((S, L, H * G, w, d)).astype(np.float32)
    k = rng.standard_normal((S, L, H, T, d)).astype(np.float32)
    v = rng.standard_normal((S, L, H, T, d)).astype(np.float32)
    inc = rng.exponential(size=(N, P - 1))
    curves = np.zeros((N, P), np.float32)
    curves[:, 1:] = np.cumsum(inc, axis=1)
    Bs = [10, 50]
    out = oracle.compress(q, k, v, curves, Bs, G, kp)
    np.testing.assert_array_equal(out["budgets"].sum(axis=1), Bs)
    assert out["offsets"][-1] == sum(Bs) + S * N * w == out["k_out"].shape[0]
    assert out["offsets"][N] == Bs[0] + N * w                  # sequence 1 starts after sequence 0
    for s_ in range(S):
        single = oracle.compress(q[s_:s_ + 1], k[s_:s_ + 1], v[s_:s_ + 1], curves, [Bs[s_]], G, kp)
        lo, hi = out["offsets"][s_ * N], out["offsets"][(s_ + 1) * N]
        np.testing.assert_array_equal(out["kept_idx"][lo:hi], single["kept_idx"])
        np.testing.assert_array_equal(out["k_out"][lo:hi], single["k_out"])
        np.testing.assert_array_equal(out["budgets"][s_], single["budgets"][0])


def test_ragged_batch_is_the_concatenation_of_single_sequence_runs(oracle):
    O = oracle
    """Sequences of different lengths in one batch (App. E): by definition one run per sequence.  With equal
    lengths the ragged form must reproduce the batched run bit for bit; with different lengths every sequence
    must be untouched by its neighbours and by the padding behind its last position."""
    rng = np.random.default_rng(12)
    S, L, H, G, d, T, w, kp, P = 3, 1, 2, 2, 8, 48, 4, 3, 9
    q = rng.standard_normal((S, L, H * G, w, d)).astype(np.float32)
    k = rng.standard_normal((S, L, H, T, d)).astype(np.float32)
    v = rng.standard_normal((S, L, H, T, d)).astype(np.float32)
    U = np.zeros((L * H, P), np.float32)
    U[:, 1:] = np.cumsum(rng.exponential(size=(L * H, P - 1)), axis=1)
    same = O.compress_ragged(q, k, v, U, [20, 31, 7], [T, T, T], G, kp)
    ref = O.compress(q, k, v, U, [20, 31, 7], G, kp)
    for key in ("k_out", "v_out", "kept_idx", "budgets", "offsets"):
        np.testing.assert_array_equal(same[key], ref[key])
    lens = [48, 32, 16]                       # each a multiple of P-1 = 8
    rag = O.compress_ragged(q, k, v, U, [20, 15, 7], lens, G, kp)
    k2, v2 = k.copy(), v.copy()
    k2[1, :, :, 32:] = 99.0                   # padding behind a sequence's last position is never read
    v2[2, :, :, 16:] = -99.0
    rag2 = O.compress_ragged(q, k2, v2, U, [20, 15, 7], lens, G, kp)
    for key in ("k_out", "v_out", "kept_idx", "budgets", "offsets"):
        np.testing.assert_array_equal(rag[key], rag2[key])
    assert rag["offsets"][-1] == 20 + 15 + 7 + S * L * H * w
    for s, Ts in enumerate(lens):
        one = O.compress(q[s:s + 1], k[s:s + 1, :, :, :Ts], v[s:s + 1, :, :, :Ts], U, [[20, 15, 7][s]], G, kp)
        np.testing.assert_array_equal(rag["budgets"][s], one["budgets"][0])
        r0, r1 = rag["offsets"][s * L * H], rag["offsets"][(s + 1) * L * H]
        np.testing.assert_array_equal(rag["kept_idx"][r0:r1], one["kept_idx"])
        assert rag["kept_idx"][r0:r1].max() == Ts - 1          # the window ends at the sequence's own last position
