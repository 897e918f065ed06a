"""Pins for the oracle's hull relaxation and greedy allocation (Sec. 4.2, App. A.2)."""
import itertools
import os

import numpy as np
import pytest
from sklearn.isotonic import IsotonicRegression

GOLD = os.path.join(os.path.dirname(__file__), "golden", "hull_hand_example.txt")


def _curves(rng, N, P, concave=False):
    inc = rng.exponential(size=(N, P - 1)) * np.where(rng.random((N, P - 1)) < 0.2, 3.0, 1.0)
    if concave:
        inc = -np.sort(-inc, axis=1)
    U = np.zeros((N, P), np.float32)
    U[:, 1:] = np.cumsum(inc, axis=1)
    return U


def _upper_hull_monotone_chain(U):
    """Least concave majorant of the points (k, U[k]) evaluated on the grid (float64)."""
    pts = [(float(k), float(u)) for k, u in enumerate(U)]
    hull = []
    for p in pts:
        while len(hull) >= 2:
            (x1, y1), (x2, y2) = hull[-2], hull[-1]
            # drop the middle point when it lies on or below the chord hull[-2] -> p
            if (y2 - y1) * (p[0] - x1) <= (p[1] - y1) * (x2 - x1):
                hull.pop()
            else:
                break
        hull.append(p)
    xs, ys = zip(*hull)
    return np.interp(np.arange(len(U)), xs, ys)


def _majorant_by_definition(U):
    P = len(U)
    out = np.array(U, np.float64)
    for k in range(P):
        for l in range(k + 1):
            for r in range(k, P):
                if r > l:
                    out[k] = max(out[k], U[l] + (U[r] - U[l]) * (k - l) / (r - l))
    return out


def test_hand_example(oracle):
    Us, Gs = [], []
    for line in open(GOLD):
        if line.startswith("U "):
            Us.append([float(x) for x in line.split()[1:]])
        elif line.startswith("G "):
            Gs.append([float(x) for x in line.split()[1:]])
    assert len(Us) == len(Gs) == 2
    for U, G in zip(Us, Gs):
        g64, g32 = oracle.hull(np.array([U], np.float32))
        np.testing.assert_allclose(g64[0], G, rtol=0, atol=1e-15)
        np.testing.assert_array_equal(g32[0], np.array(G, np.float32))


@pytest.mark.parametrize("seed", range(5))
def test_pava_matches_library_isotonic_regression(oracle, seed):
    rng = np.random.default_rng(seed)
    U = _curves(rng, 6, 40)
    g64, g32 = oracle.hull(U)
    for h in range(U.shape[0]):
        inc = np.diff(U[h].astype(np.float64))
        iso = IsotonicRegression(increasing=False).fit_transform(np.arange(len(inc)), inc)
        np.testing.assert_allclose(g64[h], np.maximum(iso, 0.0), rtol=1e-9, atol=1e-12)
    np.testing.assert_array_equal(g32, g64.astype(np.float32))


@pytest.mark.parametrize("seed", range(4))
def test_hull_properties(oracle, seed):
    rng = np.random.default_rng(100 + seed)
    N, P = 5, 24
    U = _curves(rng, N, P)
    if seed == 3:                                    # curves with dips (negative increments)
        U = (U - 0.9 * np.arange(P, dtype=np.float32)[None, :]).astype(np.float32)
    g64, _ = oracle.hull(U)
    for h in range(N):
        g = g64[h]
        assert np.all(g >= 0.0)
        assert np.all(np.diff(g) <= 0.0)                      # non-increasing (Eq. marginal_gain)
        maj = _majorant_by_definition(U[h].astype(np.float64))
        chain = _upper_hull_monotone_chain(U[h].astype(np.float64))
        np.testing.assert_allclose(chain, maj, rtol=1e-12, atol=1e-12)
        # slopes of the majorant, clipped at 0, are the gains; the telescoping identity of
        # App. A.2 rebuilds the surrogate from them
        np.testing.assert_allclose(g, np.maximum(np.diff(maj), 0.0), rtol=1e-9, atol=1e-12)
        if np.all(np.diff(maj) >= 0):
            rebuilt = U[h, 0] + np.concatenate([[0.0], np.cumsum(g)])
            np.testing.assert_allclose(rebuilt, maj, rtol=1e-9, atol=1e-9)
            assert np.all(rebuilt >= U[h].astype(np.float64) - 1e-9)
            assert abs(rebuilt[-1] - U[h, -1]) < 1e-9 and rebuilt[0] == U[h, 0]


def test_concave_curve_is_a_fixed_point_and_hull_is_idempotent(oracle):
    rng = np.random.default_rng(7)
    U = _curves(rng, 4, 30, concave=True)
    g64, _ = oracle.hull(U)
    np.testing.assert_allclose(g64, np.diff(U.astype(np.float64), axis=1), rtol=1e-12)
    V = _curves(rng, 4, 30)
    g1, _ = oracle.hull(V)
    W = np.zeros_like(V, dtype=np.float64)
    W[:, 1:] = np.cumsum(g1, axis=1)
    g2, _ = oracle.hull(W.astype(np.float32))
    np.testing.assert_allclose(g2, g1, rtol=1e-5)


# ---- greedy --------------------------------------------------------------------------------

def _pw_value(knots, b, s):
    """Piecewise-linear interpolation of curve points (grid step s tokens) at b tokens."""
    k, r = divmod(b, s)
    if r == 0:
        return knots[k]
    return knots[k] + (knots[k + 1] - knots[k]) * r / s


def _exhaustive_best(curves64, T, w, B):
    N, P = curves64.shape
    s, n = T // (P - 1), T - w
    best = -np.inf
    for split in itertools.product(range(n + 1), repeat=N - 1):
        last = B - sum(split)
        if 0 <= last <= n:
            val = sum(_pw_value(curves64[h], b, s) for h, b in enumerate(split + (last,)))
            best = max(best, val)
    return best


def _hull_curves(oracle, U):
    g64, _ = oracle.hull(U)
    H = np.zeros(U.shape, np.float64)
    H[:, 0] = U[:, 0]
    H[:, 1:] = U[:, :1] + np.cumsum(g64, axis=1)
    return H


@pytest.mark.parametrize("seed", range(6))
def test_greedy_on_concave_curves_matches_exhaustive_search(oracle, seed):
    rng = np.random.default_rng(200 + seed)
    N, P, T, w = 3, 5, 12, 2          # s = 3, n = 10
    U = _curves(rng, N, P, concave=True)
    for B in (0, 1, 7, 13, 22, N * (T - w)):
        b, off = oracle.allocate(U, T, w, [B])
        assert b.sum() == B and b.min() >= 0 and b.max() <= T - w
        val = sum(_pw_value(U[h].astype(np.float64), int(b[0, h]), T // (P - 1)) for h in range(N))
        best = _exhaustive_best(U.astype(np.float64), T, w, B)
        assert abs(val - best) <= 1e-9 * max(1.0, abs(best))


@pytest.mark.parametrize("seed", range(6))
def test_greedy_on_nonconcave_curves_matches_exhaustive_search_over_hull(oracle, seed):
    rng = np.random.default_rng(300 + seed)
    N, P, T, w = 3, 7, 12, 1          # s = 2, n = 11
    U = _curves(rng, N, P)
    Hc = _hull_curves(oracle, U)
    s = T // (P - 1)
    for B in (0, 3, 8, 16, 25, N * (T - w)):
        b, _ = oracle.allocate(U, T, w, [B])
        assert b.sum() == B
        val_hull = sum(_pw_value(Hc[h], int(b[0, h]), s) for h in range(N))
        best_hull = _exhaustive_best(Hc, T, w, B)
        assert abs(val_hull - best_hull) <= 1e-6 * max(1.0, abs(best_hull))
        # the relaxation bounds the raw problem from above (hull >= curve)
        best_raw = _exhaustive_best(U.astype(np.float64), T, w, B)
        assert best_hull >= best_raw - 1e-6


def test_budget_sum_nestedness_and_offsets(oracle):
    rng = np.random.default_rng(5)
    N, P, T, w = 16, 33, 1024, 16
    U = _curves(rng, N, P)
    n = T - w
    Bs = [0, 1, 777, 4000, 9000, N * n]
    b, off = oracle.allocate(U, T, w, Bs)
    assert b.shape == (len(Bs), N)
    np.testing.assert_array_equal(b.sum(axis=1), Bs)
    assert np.all(np.diff(b, axis=0) >= 0)                 # larger budget never shrinks a head
    assert np.all(b[-1] == n) and np.all(b[0] == 0)
    flat = (b + w).reshape(-1)
    np.testing.assert_array_equal(off, np.concatenate([[0], np.cumsum(flat)]))


def test_budgets_sit_on_hull_vertices_except_at_threshold(oracle):
    rng = np.random.default_rng(6)
    N, P, T, w = 12, 17, 512, 8
    U = _curves(rng, N, P)
    s, n = T // (P - 1), T - w
    g64, g32 = oracle.hull(U)
    b, _ = oracle.allocate(U, T, w, [1500])
    partial = 0
    for h in range(N):
        bh = int(b[0, h])
        if bh in (0, n):
            continue
        k, r = divmod(bh, s)
        if r != 0:
            partial += 1
            continue
        # a fully-bought prefix of segments: either ends at a gain drop (hull vertex) or at the
        # threshold gain shared with other heads
        assert g32[h, k - 1] >= g32[h, k]
    assert partial <= 1


def test_identical_strictly_concave_curves_give_uniform_budgets(oracle):
    N, P, T, w = 6, 9, 64, 8
    inc = np.array([8, 7, 6, 5, 4, 3, 2, 1], np.float64)
    U = np.zeros((N, P), np.float32)
    U[:, 1:] = np.cumsum(inc)[None, :]
    s = T // (P - 1)
    for segs in (1, 3, 5):
        b, _ = oracle.allocate(U, T, w, [N * s * segs])
        assert np.all(b == s * segs)


def test_tie_rule_lowest_segment_then_lowest_head(oracle):
    # flat gains everywhere: order is (k asc, hid asc); the marginal item is taken partially
    N, P, T, w = 3, 5, 16, 2          # s = 4, n = 14 -> caps 4,4,4,2
    U = np.tile(np.arange(P, dtype=np.float32), (N, 1))
    b, _ = oracle.allocate(U, T, w, [4 + 4 + 3])
    np.testing.assert_array_equal(b[0], [4, 4, 3])
    b, _ = oracle.allocate(U, T, w, [12 + 5])
    np.testing.assert_array_equal(b[0], [8, 5, 4])
    b, _ = oracle.allocate(U, T, w, [36 + 3])          # last segments hold only 2 tokens
    np.testing.assert_array_equal(b[0], [14, 13, 12])


def test_zero_gain_segments_are_taken_last_and_budget_errors(oracle):
    N, P, T, w = 2, 3, 8, 2           # s = 4, n = 6 -> caps 4,2
    U = np.array([[0, 5, 5], [0, 1, 0.5]], np.float32)   # head 1's tail decreases -> gain 0
    b, _ = oracle.allocate(U, T, w, [9])
    np.testing.assert_array_equal(b[0], [5, 4])           # zero-gain items: k=1 of head 0 first
    with pytest.raises(ValueError):
        oracle.allocate(U, T, w, [13])
    with pytest.raises(ValueError):
        oracle.allocate(U, T, w, [-1])
