"""Pins for the oracle's exact allocation solver (Sec. 4.2, Eq. "combinatorial_optimization")."""
import itertools

import numpy as np


def _curves(rng, N, P, concave=False):
    inc = rng.exponential(size=(N, P - 1)) * np.where(rng.random((N, P - 1)) < 0.2, 3.0, 1.0)
    if concave:
        inc = -np.sort(-inc, axis=1)
    U = np.zeros((N, P), np.float32)
    U[:, 1:] = np.cumsum(inc, axis=1)
    return U


def _value(U, b):
    return float(sum(np.float64(U[h, int(b[h])]) for h in range(U.shape[0])))


def test_exact_against_exhaustive_search(oracle):
    rng = np.random.default_rng(70)
    N, T, w = 3, 9, 2
    n = T - w
    for trial in range(4):
        U = _curves(rng, N, T + 1)
        U[:, 1:] -= rng.random((N, T)).astype(np.float32) * 0.5          # not even monotone
        for B in (0, 1, 5, 11, N * n):
            b, val = oracle.exact_allocate(U, T, w, [B])
            best = max(_value(U, split + (B - sum(split),))
                       for split in itertools.product(range(n + 1), repeat=N - 1) if 0 <= B - sum(split) <= n)
            assert abs(val[0] - best) <= 1e-12 * max(1.0, abs(best))
            assert b.sum() == B and b.min() >= 0 and b.max() <= n
            assert abs(_value(U, b[0]) - best) <= 1e-12 * max(1.0, abs(best))


def test_exact_equals_greedy_on_concave_curves(oracle):
    # App. A.2: on concave curves the marginal-utility greedy is optimal
    rng = np.random.default_rng(71)
    N, T, w = 6, 40, 4
    U = _curves(rng, N, T + 1, concave=True)
    for B in (0, 7, 50, 133, N * (T - w)):
        bg, _ = oracle.allocate(U, T, w, [B])
        _, val = oracle.exact_allocate(U, T, w, [B])
        assert abs(_value(U, bg[0]) - val[0]) <= 1e-9 * max(1.0, val[0])


def test_exact_lies_between_the_greedy_and_its_relaxation(oracle):
    # raw value of the greedy's budgets <= exact optimum on the raw curves <= optimum of the relaxed (hull) problem
    rng = np.random.default_rng(72)
    N, T, w = 8, 64, 8
    U = _curves(rng, N, T + 1)
    g64, _ = oracle.hull(U)
    Hc = np.concatenate([np.zeros((N, 1)), np.cumsum(g64, axis=1)], axis=1)
    gaps = []
    for B in (10, 100, 224, 400):
        bg, _ = oracle.allocate(U, T, w, [B])
        _, val = oracle.exact_allocate(U, T, w, [B])
        raw = _value(U, bg[0])
        relaxed = float(sum(Hc[h, int(bg[0, h])] for h in range(N)))
        assert raw <= val[0] + 1e-9 and val[0] <= relaxed + 1e-6
        gaps.append(val[0] - raw)
    assert max(gaps) > 0          # rough curves: the relaxation does lose something somewhere


def test_batch_and_errors(oracle):
    import pytest
    rng = np.random.default_rng(73)
    U = _curves(rng, 4, 21)
    b, val = oracle.exact_allocate(U, 20, 4, [0, 9, 64])
    assert list(b.sum(axis=1)) == [0, 9, 64] and val[0] == 0.0 and (b[2] == 16).all()
    assert val[1] <= val[2]
    with pytest.raises(ValueError):
        oracle.exact_allocate(U, 20, 4, [65])
    with pytest.raises(ValueError):
        oracle.exact_allocate(_curves(rng, 4, 11), 20, 4, [5])     # not token resolution
