"""Pins for the oracle's curve builder (Sec. 3.2 M^pi(k); Eq. "head_loss_def")."""
import numpy as np


def test_curve_is_the_importance_mass_of_the_selected_set(oracle):
    # U(k) must equal the importance of exactly the positions the (separately pinned) selection keeps
    rng = np.random.default_rng(1)
    heads, T, w, P = 3, 48, 6, 9           # s = 6, n = 42: the last point is clipped at n
    n = T - w
    scores = rng.random((heads, n)).astype(np.float32)
    scores[1, 5:15] = scores[1, 5]         # ties
    imp = rng.random((heads, n)).astype(np.float32)
    for n_sink in (0, 4):
        U = oracle.build_curves(scores, imp, T, w, P, n_sink=n_sink)
        for u in range(heads):
            for k in range(P):
                b = min(k * (T // (P - 1)), n)
                kept = oracle.select(scores[u], b, n_sink=n_sink)
                want = np.float32(imp[u][kept].astype(np.float64).sum())
                assert abs(float(U[u, k]) - float(want)) <= 2e-7 * max(1.0, float(want)), (u, k)
        # total loss L(empty set) = all the importance: the last point
        np.testing.assert_allclose(U[:, -1], imp.astype(np.float64).sum(axis=1), rtol=2e-7)
        assert (U[:, 0] == 0).all() and (np.diff(U.astype(np.float64), axis=1) >= 0).all()


def test_uniform_importance_gives_a_straight_line(oracle):
    heads, T, w, P = 2, 64, 8, 17
    n = T - w
    scores = np.random.default_rng(2).random((heads, n)).astype(np.float32)
    U = oracle.build_curves(scores, np.ones((heads, n), np.float32), T, w, P)
    np.testing.assert_array_equal(U, np.broadcast_to(np.minimum(np.arange(P) * 4, n).astype(np.float32), U.shape))


def test_oracle_metric_gives_the_concave_top_k_curve(oracle):
    # ranking by the importance itself (the oracle metric of Sec. 3.2): U(k) is the sum of the k largest
    # values, its increments never grow, and the hull relaxation leaves it unchanged
    rng = np.random.default_rng(3)
    heads, T, w, P = 4, 256, 0 + 16, 33
    n = T - w
    imp = rng.exponential(size=(heads, n)).astype(np.float32)
    U = oracle.build_curves(imp, imp, T, w, P)
    s = T // (P - 1)
    top = -np.sort(-imp.astype(np.float64), axis=1)
    want = np.concatenate([np.zeros((heads, 1)), np.cumsum(top, axis=1)], axis=1)[:, np.minimum(np.arange(P) * s, n)]
    np.testing.assert_allclose(U, want, rtol=2e-7)
    inc = np.diff(U.astype(np.float64), axis=1)
    assert (np.diff(inc[:, :-1], axis=1) <= 1e-4).all()          # the last segment is clipped
    g64, _ = oracle.hull(U)
    np.testing.assert_allclose(g64[:, :-1], inc[:, :-1], rtol=1e-5, atol=1e-6)


def test_a_worse_ranking_never_beats_the_oracle_ranking(oracle):
    rng = np.random.default_rng(4)
    heads, T, w, P = 3, 128, 8, 17
    n = T - w
    imp = rng.exponential(size=(heads, n)).astype(np.float32)
    noisy = (imp * rng.lognormal(sigma=1.0, size=imp.shape)).astype(np.float32)
    best = oracle.build_curves(imp, imp, T, w, P).astype(np.float64)
    got = oracle.build_curves(noisy, imp, T, w, P).astype(np.float64)
    assert (got <= best + 1e-4).all() and (got[:, 1:-1] < best[:, 1:-1]).any()
    np.testing.assert_allclose(got[:, -1], best[:, -1], rtol=1e-6)   # everything kept: nothing lost either way
