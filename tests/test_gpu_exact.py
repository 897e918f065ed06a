"""GPU parity of the exact allocation solver (Sec. 4.2, Eq. "combinatorial_optimization") against the oracle.
The optimum is unique, the optimal budgets need not be: the optimum is compared (fp32 accumulation over N
heads against the oracle's fp64: relative 1e-5), the budgets are checked to be feasible and to reach it."""
import numpy as np
import pytest
import torch

from paper_2602_08585_b200 import lukv, synth

pytestmark = pytest.mark.gpu
RTOL = 1e-5


def gpu_exact(N, T, w, U, Bs, L=1):
    p = lukv.make_params(len(Bs), L, N // L, 1, 64, T, w, 1, "fp32", T + 1)
    ws = torch.empty(lukv.lukv_exact_workspace_bytes(p, max(Bs)), dtype=torch.uint8, device="cuda")
    budgets = torch.full((len(Bs), N), -7, dtype=torch.int32, device="cuda")
    offsets = torch.full((len(Bs) * N + 1,), -7, dtype=torch.int32, device="cuda")
    values = torch.zeros(len(Bs), dtype=torch.float64, device="cuda")
    lukv.lukv_exact_allocate(p, torch.from_numpy(np.ascontiguousarray(U, np.float32)).cuda(), Bs, budgets, offsets,
                             values, ws)
    torch.cuda.synchronize()
    return budgets.cpu().numpy(), offsets.cpu().numpy(), values.cpu().numpy()


def _value(U, b):
    return float(np.take_along_axis(U.astype(np.float64), b.astype(np.int64)[:, None], axis=1).sum())


def _check(oracle, N, T, w, U, Bs, L=1):
    n = T - w
    b, off, val = gpu_exact(N, T, w, U, Bs, L)
    _, val_ref = oracle.exact_allocate(U, T, w, Bs)
    for q, B in enumerate(Bs):
        tol = RTOL * max(1.0, abs(val_ref[q]))
        assert abs(val[q] - val_ref[q]) <= tol, (q, val[q], val_ref[q])
        assert b[q].sum() == B and b[q].min() >= 0 and b[q].max() <= n
        assert abs(_value(U, b[q]) - val_ref[q]) <= tol
    np.testing.assert_array_equal(off, np.concatenate([[0], np.cumsum(b.reshape(-1) + w)]))


def _rough(rng, N, P):
    inc = rng.exponential(size=(N, P - 1)) * np.where(rng.random((N, P - 1)) < 0.2, 3.0, 1.0)
    U = np.zeros((N, P), np.float32)
    U[:, 1:] = np.cumsum(inc, axis=1)
    return U


def test_small_cases_and_edges(oracle):
    rng = np.random.default_rng(80)
    N, T, w = 5, 40, 4
    U = _rough(rng, N, T + 1)
    U[:, 1:] -= rng.random((N, T)).astype(np.float32)            # not monotone
    _check(oracle, N, T, w, U, [0, 1, 17, 36, 100, N * (T - w) - 1, N * (T - w)])
    _check(oracle, 1, 16, 3, _rough(rng, 1, 17), [0, 5, 13])       # one head: b = B
    _check(oracle, 3, 8, 7, _rough(rng, 3, 9), [0, 2, 3])          # one rankable position per head


def test_medium_size_spans_many_tiles(oracle):
    rng = np.random.default_rng(81)
    N, T, w = 64, 1024, 32                                          # n = 992; budgets beyond one tile of 1024
    U = synth.gen_calibration_curves(81, 1, N, T)[0]
    _check(oracle, N, T, w, U, [5000, 30000], L=8)


def test_calibration_size_sandwich(oracle):
    # 256 heads x 3968 tokens: the oracle's recursion would take minutes; instead
    # value(greedy budgets on the raw curves) <= exact optimum <= optimum of the relaxed problem
    N, T, w = 256, 4000, 32
    n = T - w
    U = synth.gen_calibration_curves(synth.BASE_SEED, 1, N, T)[0]
    B = int(0.3 * N * n)
    b, off, val = gpu_exact(N, T, w, U, [B], L=32)
    assert b[0].sum() == B and b[0].min() >= 0 and b[0].max() <= n
    assert abs(_value(U, b[0]) - val[0]) <= RTOL * val[0]
    bg, _ = oracle.allocate(U, T, w, [B])
    g64, _ = oracle.hull(U)
    Hc = np.concatenate([np.zeros((N, 1)), np.cumsum(g64, axis=1)], axis=1)
    raw = _value(U, bg[0])
    relaxed = float(np.take_along_axis(Hc, bg[0].astype(np.int64)[:, None], axis=1).sum())
    assert raw <= val[0] * (1 + RTOL) and val[0] <= relaxed * (1 + RTOL)
    # the paper's point: the relaxation gives up very little
    assert (val[0] - raw) / val[0] < 0.01


def test_unsupported_shapes():
    f = torch.empty(1, device="cuda")
    p = lukv.make_params(1, 1, 4, 1, 64, 64, 8, 1, "fp32", 33)      # 2 tokens per segment
    assert lukv.lukv_exact_allocate(p, f, [10], f, f, f, f, check=False) == lukv.ERR_UNSUPPORTED
    p = lukv.make_params(1, 1, 4, 1, 64, 64, 8, 1, "fp32", 65, min_keep=0.1)
    assert lukv.lukv_exact_allocate(p, f, [40], f, f, f, f, check=False) == lukv.ERR_UNSUPPORTED
