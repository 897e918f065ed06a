"""GPU parity of the KeyDiff proxy (pi_2 of Sec. 5.1) against the oracle, and the path built on it: KeyDiff scores
-> per-head top-b selection and gather with the recent window of 1 that App. E uses for this metric.
The scores are cosines in [-1, 1] from fp32 sums over d channels and T keys: absolute tolerance 2e-5 (the anchor
is a mean of T unit vectors accumulated in fp32 in slices of a few hundred keys; the dot products add d terms)."""
import numpy as np
import pytest
import torch

from paper_2602_08585_b200 import lukv
from gpu_helpers import bits, gpu_select_gather

pytestmark = pytest.mark.gpu
ATOL = 2e-5


def gpu_keydiff(p, k):
    ws = lukv.alloc_workspace(p)
    scores = torch.full((p.batch, p.N, p.n), -7.0, dtype=torch.float32, device="cuda")
    status = torch.full((1,), 5, dtype=torch.int32, device="cuda")
    lukv.lukv_score_keydiff(p, k.cuda(), scores, ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return scores


SHAPES = [
    # S, L, H, d,   T,    w, dtype
    (1, 1, 1, 64, 2, 1, torch.float32),            # smallest legal problem
    (2, 1, 3, 64, 77, 1, torch.bfloat16),          # ragged, 8 lanes per key row
    (1, 2, 2, 128, 1300, 1, torch.bfloat16),       # several chunks, ragged tail
    (1, 1, 2, 128, 1025, 5, torch.float32),        # 32 lanes per key row, wider window
    (1, 1, 3, 64, 4096 + 33, 33, torch.float32),
    (1, 4, 8, 128, 16384, 1, torch.bfloat16),      # more heads than one L2 group of keys holds at this length
    (2, 4, 8, 64, 300, 7, torch.bfloat16),         # many short heads: slices that span several heads
    (1, 2, 5, 128, 64 * 37 + 1, 1, torch.float32), # one row past a whole number of stages
]


@pytest.mark.parametrize("shape", SHAPES)
def test_keydiff_matches_oracle(oracle, shape):
    S, L, H, d, T, w, dtype = shape
    g = torch.Generator().manual_seed(T + d)
    k = (torch.randn((S, L, H, T, d), generator=g) * torch.rand((S, L, H, T, 1), generator=g) * 4.0 + 0.3).to(dtype)
    k[0, 0, 0, 0] = 0                                 # a zero key scores 0
    p = lukv.make_params(S, L, H, 1, d, T, w, 1, dtype, 2)
    got = gpu_keydiff(p, k).cpu().numpy()
    ref = oracle.keydiff(bits(k), w)
    np.testing.assert_allclose(got, ref, rtol=0, atol=ATOL)
    assert got[0, 0, 0] == 0.0


@pytest.mark.parametrize("group_mb", [1, 2, 3])
def test_keydiff_many_groups(oracle, monkeypatch, group_mb):
    """Groups of one to three heads (the group size is a tuning switch): every CTA alternates many times between
    summing one group and scoring the one before it, and the last group is smaller than the others."""
    monkeypatch.setenv("LUKV_KEYDIFF_GROUP_MB", str(group_mb))
    S, L, H, d, T, w = 1, 1, 7, 128, 4096, 1          # 1 MB of bf16 keys per head
    g = torch.Generator().manual_seed(group_mb)
    k = (torch.randn((S, L, H, T, d), generator=g) + 0.5).to(torch.bfloat16)
    p = lukv.make_params(S, L, H, 1, d, T, w, 1, torch.bfloat16, 2)
    got = gpu_keydiff(p, k).cpu().numpy()
    np.testing.assert_allclose(got, oracle.keydiff(bits(k), w), rtol=0, atol=ATOL)


def test_keydiff_wait_runs_out(monkeypatch):
    """A head whose anchor is never published (a host-side switch of the library drops the publication): the CTAs
    that score it give up after the bounded wait, the call reports LUKV_ERR_TIMEOUT in dev_status, the device stays
    usable and the next call is correct."""
    S, L, H, d, T, w = 1, 1, 4, 128, 2048, 1
    g = torch.Generator().manual_seed(5)
    k = torch.randn((S, L, H, T, d), generator=g).to(torch.bfloat16).cuda()
    p = lukv.make_params(S, L, H, 1, d, T, w, 1, torch.bfloat16, 2)
    ws = lukv.alloc_workspace(p)
    scores = torch.empty((S, L * H, T - w), dtype=torch.float32, device="cuda")
    status = torch.zeros((1,), dtype=torch.int32, device="cuda")

    def call():
        lukv.lukv_score_keydiff(p, k, scores, ws, status)
        torch.cuda.synchronize()
        return int(status.item())

    assert call() == 0
    good = scores.clone()
    monkeypatch.setenv("LUKV_TEST_SPIN_LIMIT", "20000")
    monkeypatch.setenv("LUKV_TEST_DROP_ITEM", "2")
    assert call() == lukv.ERR_TIMEOUT
    monkeypatch.delenv("LUKV_TEST_SPIN_LIMIT")
    monkeypatch.delenv("LUKV_TEST_DROP_ITEM")
    assert call() == 0
    assert torch.equal(scores, good)


def test_keydiff_selection_and_gather(oracle):
    """The deployed combination of App. E: KeyDiff scores, recent window 1, per-head top-b."""
    S, L, H, d, T, w = 1, 2, 3, 128, 3000, 1
    g = torch.Generator().manual_seed(3)
    k = torch.randn((S, L, H, T, d), generator=g).to(torch.bfloat16)
    v = torch.randn((S, L, H, T, d), generator=g).to(torch.bfloat16)
    p = lukv.make_params(S, L, H, 1, d, T, w, 1, torch.bfloat16, 2)
    scores = gpu_keydiff(p, k)
    ref_scores = oracle.keydiff(bits(k), w)
    N, n = L * H, T - w
    budgets = np.array([[0, 1, n // 5, n // 2, n - 1, n]], np.int32)
    offsets = np.concatenate([[0], np.cumsum(budgets.reshape(-1) + w)]).astype(np.int32)
    rows = int(offsets[-1])
    # selection and gather on the oracle's scores: bit-exact
    k_out, v_out, kept = gpu_select_gather(p, torch.from_numpy(ref_scores).cuda(), torch.from_numpy(budgets).cuda(),
                                           torch.from_numpy(offsets).cuda(), k.cuda(), v.cuda(), rows)
    rk, rv, rkept = oracle.select_gather(ref_scores.reshape(N, n), budgets, offsets, bits(k).reshape(N, T, d),
                                         bits(v).reshape(N, T, d), w)
    np.testing.assert_array_equal(kept.cpu().numpy()[:rows], rkept)
    np.testing.assert_array_equal(bits(k_out)[:rows], rk)
    # on the GPU's own scores: the same sets up to positions whose scores tie within the tolerance
    _, _, kept2 = gpu_select_gather(p, scores, torch.from_numpy(budgets).cuda(), torch.from_numpy(offsets).cuda(),
                                    k.cuda(), v.cuda(), rows)
    kept2 = kept2.cpu().numpy()
    same = total = 0
    for u in range(N):
        b, o = budgets.reshape(-1)[u], offsets[u]
        if b == 0:
            continue
        a, r = kept2[o:o + b], rkept[o:o + b]
        same += len(np.intersect1d(a, r))
        total += b
        diff = np.setxor1d(a, r)
        if len(diff):
            t = np.sort(ref_scores.reshape(N, n)[u])[::-1][b - 1]
            assert np.all(np.abs(ref_scores.reshape(N, n)[u][diff] - t) <= 2 * ATOL)
        assert kept2[o + b] == n                      # the recent window of one position
    assert same / total >= 0.999
