"""Pins for the oracle's deployment settings of App. E: attention sinks and the minimum retention per head."""
import itertools

import numpy as np
import pytest


def _curves(rng, N, P, concave=False):
    inc = rng.exponential(size=(N, P - 1)) * np.where(rng.random((N, P - 1)) < 0.2, 3.0, 1.0)
    if concave:
        inc = -np.sort(-inc, axis=1)
    U = np.zeros((N, P), np.float32)
    U[:, 1:] = np.cumsum(inc, axis=1)
    return U


def _pw_value(curve, b, s):
    """Piecewise-linear utility of keeping b tokens (curve points every s tokens)."""
    k, r = divmod(b, s)
    if r == 0:
        return curve[k]
    return curve[k] + (curve[k + 1] - curve[k]) * r / s


def _best_with_floor(curves64, T, w, B, f):
    N, P = curves64.shape
    s, n = T // (P - 1), T - w
    best = -np.inf
    for split in itertools.product(range(f, n + 1), repeat=N - 1):
        last = B - sum(split)
        if f <= last <= n:
            best = max(best, sum(_pw_value(curves64[h], b, s) for h, b in enumerate(split + (last,))))
    return best


def test_floor_tokens(oracle):
    assert oracle.floor_tokens(0.0, 1000) == 0
    assert oracle.floor_tokens(0.01, 1000) == 10          # float32(0.01) is a little below 0.01
    assert oracle.floor_tokens(0.01, 32736) == 328         # 327.36 rounds up
    assert oracle.floor_tokens(0.5, 7) == 4
    assert oracle.floor_tokens(1.0, 7) == 7
    assert oracle.floor_tokens(0.2, 10) == 3               # float32(0.2) is a little above 1/5: the ceiling sees it


@pytest.mark.parametrize("seed", range(5))
def test_floor_allocation_matches_constrained_exhaustive_search(oracle, seed):
    rng = np.random.default_rng(900 + seed)
    N, P, T, w = 3, 5, 12, 2          # s = 3, n = 10; the floor of 2 tokens cuts into the first segment
    U = _curves(rng, N, P, concave=True)
    min_keep = 0.125                  # exact in binary: ceil(1.25) = 2
    f = oracle.floor_tokens(min_keep, T - w)
    assert f == 2
    for B in (N * f, N * f + 1, 11, 17, 25, N * (T - w)):
        b, off = oracle.allocate(U, T, w, [B], min_keep=min_keep)
        assert b.sum() == B and b.min() >= f and b.max() <= T - w
        val = sum(_pw_value(U[h].astype(np.float64), int(b[0, h]), T // (P - 1)) for h in range(N))
        best = _best_with_floor(U.astype(np.float64), T, w, B, f)
        assert abs(val - best) <= 1e-9 * max(1.0, abs(best))
        np.testing.assert_array_equal(off, np.concatenate([[0], np.cumsum(b.reshape(-1) + w)]))
    with pytest.raises(ValueError):
        oracle.allocate(U, T, w, [N * f - 1], min_keep=min_keep)


def test_floor_is_inactive_when_the_plain_solution_already_satisfies_it(oracle):
    rng = np.random.default_rng(12)
    N, P, T, w = 10, 33, 1024, 16
    U = _curves(rng, N, P)
    n = T - w
    Bs = [2000, 5000, 9000, N * n]
    plain, _ = oracle.allocate(U, T, w, Bs)
    for q, B in enumerate(Bs):
        f = int(plain[q].min())
        mk = np.float32(f / n)
        while oracle.floor_tokens(float(mk), n) > f:          # a ratio whose ceiling is exactly f
            mk = np.nextafter(mk, np.float32(0))
        if oracle.floor_tokens(float(mk), n) != f:
            continue
        got, _ = oracle.allocate(U, T, w, [B], min_keep=float(mk))
        np.testing.assert_array_equal(got[0], plain[q])


def test_floor_raises_starved_heads_and_keeps_the_sum(oracle):
    rng = np.random.default_rng(13)
    N, P, T, w = 8, 17, 512, 8
    U = _curves(rng, N, P)
    U[3] *= 1e-3                                              # a head nobody would buy from
    n = T - w
    B = N * n // 10
    plain, _ = oracle.allocate(U, T, w, [B])
    assert plain[0, 3] == 0
    got, _ = oracle.allocate(U, T, w, [B], min_keep=0.01)
    f = oracle.floor_tokens(0.01, n)
    assert got.sum() == B and got.min() >= f and got[0, 3] == f
    # the others give up exactly what the floor hands out, never more than they had
    assert (got[0] <= np.maximum(plain[0], f)).all()


def test_sinks_rank_first(oracle):
    rng = np.random.default_rng(3)
    n = 50
    s = rng.random(n).astype(np.float32)
    s[:4] = 0.0                                               # the sinks have the lowest scores
    for b in (0, 2, 4, 5, 17, n):
        kept = oracle.select(s, b, n_sink=4)
        forced = list(range(min(4, b)))
        rest = sorted(np.argsort(-s[4:], kind="stable")[:max(0, b - 4)] + 4)
        assert list(kept) == forced + rest
    # without sinks the same budget keeps none of them
    assert not set(oracle.select(s, 17)) & {0, 1, 2, 3}
    # n_sink = 0 is the plain selection
    np.testing.assert_array_equal(oracle.select(s, 17, n_sink=0), oracle.select(s, 17))


def test_profile_with_floor(oracle):
    rng = np.random.default_rng(21)
    Mq, N, T, w, P = 3, 6, 128, 8, 33
    n = T - w
    U = np.stack([_curves(rng, N, P) for _ in range(Mq)])
    U[:, 2] *= 1e-3
    ratios = np.linspace(0.0, 1.0, 21).astype(np.float32)
    phi = oracle.profile_build(U, T, w, ratios, min_keep=0.05).astype(np.float64)
    f = oracle.floor_tokens(0.05, n)
    # no head is compressed beyond 1 - f/n, and at rho = 1 every head sits exactly there
    assert (phi <= 1.0 - f / n + 1e-7).all()
    np.testing.assert_allclose(phi[-1], 1.0 - f / n, rtol=0, atol=1e-7)
    # where the budget allows it the mean retained fraction still matches the global ratio
    B = np.maximum(np.floor((1.0 - ratios.astype(np.float64)) * N * n), N * f)
    np.testing.assert_allclose(((1.0 - phi) * n).sum(axis=1), B, rtol=0, atol=N * n * 1e-7)
    # lookup: budgets never fall below the floor of the new context
    Tn = 1000
    b, off = oracle.profile_budgets(phi.astype(np.float32), ratios, Tn, w, [0.3, 0.97, 1.0], min_keep=0.05)
    fn = oracle.floor_tokens(0.05, Tn - w)
    assert b.min() >= fn
    plain, _ = oracle.profile_budgets(phi.astype(np.float32), ratios, Tn, w, [0.3, 0.97, 1.0])
    np.testing.assert_array_equal(b, np.maximum(plain, fn))
    # a profile built without the floor compresses to zero at sigma = 1; the lookup's own floor lifts it
    phi0 = oracle.profile_build(U, T, w, ratios)
    b0, _ = oracle.profile_budgets(phi0, ratios, Tn, w, [1.0], min_keep=0.05)
    assert (b0 == fn).all()
