"""Pins for the oracle's offline profile and online lookup/budgeting (Sec. 4.3, Eq. "calibration_avg")."""
import os

import numpy as np
import pytest

GOLD = os.path.join(os.path.dirname(__file__), "golden", "profile_lookup_hand_example.txt")


def _concave_curves(rng, Mq, N, P):
    inc = -np.sort(-rng.exponential(size=(Mq, N, P - 1)), axis=2)
    U = np.zeros((Mq, N, P), np.float64)
    U[:, :, 1:] = np.cumsum(inc, axis=2)
    return U.astype(np.float32)


def _rough_curves(rng, Mq, N, P):
    inc = rng.exponential(size=(Mq, N, P - 1)) * np.where(rng.random((Mq, N, P - 1)) < 0.2, 3.0, 1.0)
    U = np.zeros((Mq, N, P), np.float64)
    U[:, :, 1:] = np.cumsum(inc, axis=2)
    return U.astype(np.float32)


def _token_by_token(U, n, B):
    """The marginal-utility greedy of Sec. 4.2 run one token at a time on concave curves at
    token resolution: the next token goes to the head whose next increment is largest."""
    N = U.shape[0]
    gain = (U[:, 1:].astype(np.float64) - U[:, :-1].astype(np.float64)).astype(np.float32)
    b = np.zeros(N, np.int64)
    for _ in range(B):
        best = None
        for h in range(N):
            if b[h] >= n:
                continue
            key = (-float(gain[h, b[h]]), int(b[h]), h)
            if best is None or key < best[0]:
                best = (key, h)
        b[best[1]] += 1
    return b


def test_profile_against_token_by_token_greedy(oracle):
    rng = np.random.default_rng(11)
    Mq, N, T, w = 3, 4, 12, 2
    n = T - w
    U = _concave_curves(rng, Mq, N, T + 1)
    ratios = np.array([0.0, 0.1, 0.25, 1.0 / 3.0, 0.5, 0.77, 0.9, 1.0], np.float32)
    phi = oracle.profile_build(U, T, w, ratios)
    assert phi.shape == (len(ratios), N)
    for j, rho in enumerate(ratios):
        B = int(np.floor((1.0 - float(rho)) * N * n))
        r = np.zeros(N)
        for i in range(Mq):
            r += 1.0 - _token_by_token(U[i], n, B) / n
        np.testing.assert_allclose(phi[j], r / Mq, rtol=0, atol=6e-8)


def test_single_query_is_the_allocation(oracle):
    rng = np.random.default_rng(5)
    N, T, w, P = 6, 64, 8, 17
    U = _rough_curves(rng, 1, N, P)
    ratios = np.linspace(0.0, 1.0, 21).astype(np.float32)
    phi = oracle.profile_build(U, T, w, ratios)
    n = T - w
    B = np.floor((1.0 - ratios.astype(np.float64)) * N * n).astype(np.int64)
    b, _ = oracle.allocate(U[0], T, w, B)
    np.testing.assert_array_equal(phi, (1.0 - b.astype(np.float64) / n).astype(np.float32))


def test_end_points_conservation_and_monotonicity(oracle):
    rng = np.random.default_rng(7)
    Mq, N, T, w, P = 5, 9, 96, 6, 33
    n = T - w
    U = _rough_curves(rng, Mq, N, P)
    ratios = np.linspace(0.0, 1.0, 41).astype(np.float32)
    phi = oracle.profile_build(U, T, w, ratios).astype(np.float64)
    # rho = 0 keeps every position of every head, rho = 1 none
    np.testing.assert_array_equal(phi[0], 0.0)
    np.testing.assert_array_equal(phi[-1], 1.0)
    assert (phi >= 0).all() and (phi <= 1).all()
    # every query spends exactly B(rho), so the averaged retained fractions still add up to it
    B = np.floor((1.0 - ratios.astype(np.float64)) * N * n)
    np.testing.assert_allclose(((1.0 - phi) * n).sum(axis=1), B, rtol=0, atol=N * n * 1e-7)
    # the greedy solutions are nested in the budget, so no head's ratio falls as rho grows
    assert (np.diff(phi, axis=0) >= -1e-7).all()
    # heads differ (the layout is [ratio][head], not the transpose)
    assert np.ptp(phi[len(ratios) // 2]) > 0.05


def test_identical_heads_closed_form(oracle):
    # every head has the same strictly concave curve at token resolution: the greedy deals the
    # tokens out level by level, so with B divisible by N each head keeps B/N and r = rho
    N, T, w = 4, 20, 4
    n = T - w
    k = np.arange(T + 1, dtype=np.float64)
    curve = np.sqrt(k).astype(np.float32)
    U = np.broadcast_to(curve, (3, N, T + 1)).copy()
    ratios = np.array([0.0, 0.25, 0.5, 0.75, 1.0], np.float32)
    phi = oracle.profile_build(U, T, w, ratios)
    np.testing.assert_array_equal(phi, np.broadcast_to(ratios[:, None], phi.shape))


def test_mean_over_queries(oracle):
    # two queries with opposite preferences: query 0 only values head 0, query 1 only head 1
    T, w = 10, 2
    n = T - w
    ramp = np.minimum(np.arange(T + 1), n).astype(np.float32)
    U = np.zeros((2, 2, T + 1), np.float32)
    U[0, 0] = ramp
    U[1, 1] = ramp
    phi = oracle.profile_build(U, T, w, np.array([0.5], np.float32))
    # B = 8: the valued head keeps all 8 positions (r = 0), the other none (r = 1); the mean is 1/2
    np.testing.assert_array_equal(phi, np.array([[0.5, 0.5]], np.float32))


def test_lookup_hand_example(oracle):
    rows = {}
    for line in open(GOLD):
        if line.startswith("#") or not line.strip():
            continue
        key, *vals = line.split()
        rows.setdefault(key, []).append([float(x) for x in vals])
    ratios = np.array(rows["ratios"][0], np.float32)
    profile = np.array(rows["profile"], np.float32)
    T, w = (int(x) for x in rows["T_w"][0])
    sigma = np.array(rows["sigma"][0], np.float32)
    want = np.array(rows["budgets"], np.int32)
    b, off = oracle.profile_budgets(profile, ratios, T, w, sigma)
    np.testing.assert_array_equal(b, want)
    np.testing.assert_array_equal(off, np.concatenate([[0], np.cumsum(want.reshape(-1) + w)]))


def test_lookup_properties(oracle):
    rng = np.random.default_rng(3)
    Mq, N, Tc, w, P = 4, 12, 128, 8, 129
    U = _rough_curves(rng, Mq, N, P)
    ratios = np.linspace(0.0, 1.0, 33).astype(np.float32)
    phi = oracle.profile_build(U, Tc, w, ratios)
    T = 1000
    n = T - w
    sigma = np.array([0.0, 0.25, 0.3, 0.51234, 0.9, 1.0], np.float32)
    b, off = oracle.profile_budgets(phi, ratios, T, w, sigma)
    assert b.min() >= 0 and b.max() <= n
    np.testing.assert_array_equal(b[0], n)
    np.testing.assert_array_equal(b[-1], 0)
    # floors lose less than one token per head against the target budget (up to the fp32 profile)
    target = (1.0 - sigma.astype(np.float64)) * N * n
    tot = b.sum(axis=1)
    assert (tot <= target + N * n * 1e-6).all() and (tot >= target - N - N * n * 1e-6).all()
    # more compression never gives a head more tokens
    assert (np.diff(b, axis=0) <= 0).all()
    # on the calibration context itself, one query, a grid ratio: the calibration budgets come back
    # up to the floor of a ratio that went through fp32
    phi1 = oracle.profile_build(U[:1], Tc, w, ratios)
    nc = Tc - w
    B = np.floor((1.0 - ratios.astype(np.float64)) * N * nc).astype(np.int64)
    b_cal, _ = oracle.allocate(U[0], Tc, w, B)
    b_back, _ = oracle.profile_budgets(phi1, ratios, Tc, w, ratios)
    d = b_cal.astype(np.int64) - b_back
    assert d.min() >= 0 and d.max() <= 1


def test_lookup_rejects_bad_grid(oracle):
    phi = np.zeros((2, 3), np.float32)
    with pytest.raises(ValueError):
        oracle.profile_budgets(phi, np.array([0.5, 0.5], np.float32), 64, 8, np.array([0.5], np.float32))
    with pytest.raises(ValueError):
        oracle.profile_budgets(phi, np.array([0.2, 0.5], np.float32), 64, 8, np.array([0.6], np.float32))
    with pytest.raises(ValueError):
        oracle.profile_build(np.zeros((1, 2, 9), np.float32), 64, 8, np.array([1.5], np.float32))
