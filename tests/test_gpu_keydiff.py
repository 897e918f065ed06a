"""GPU parity of the KeyDiff proxy (pi_2 of Sec. 5.1) against the oracle, and the path built on it: KeyDiff scores
-> per-head top-b selection and gather with the recent window of 1 that App. E uses for this metric.
The scores are cosines in [-1, 1] from fp32 sums over d channels and T keys: absolute tolerance 2e-5 (the anchor
is a mean of T unit vectors accumulated in fp32 in slices of a few hundred keys; the dot products add d terms)."""
import numpy as np
import pytest
import torch

from paper_2602_08585_b200 import lukv, synth
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


def _kept_close(kept_gpu, kept_ref, budgets, offsets, ref_scores, w):
    """Same kept sets, up to positions whose oracle scores lie within the tolerance of the head's threshold."""
    n = ref_scores.shape[-1]
    flat = ref_scores.reshape(-1, n)
    same = total = 0
    for u, b in enumerate(budgets.reshape(-1)):
        o = offsets[u]
        assert np.array_equal(kept_gpu[o + b:o + b + w], np.arange(n, n + w))      # the recent window
        if b == 0:
            continue
        a, r = kept_gpu[o:o + b], kept_ref[o:o + b]
        assert np.all(np.diff(a) > 0)
        same += len(np.intersect1d(a, r))
        total += b
        diff = np.setxor1d(a, r)
        if len(diff):
            t = np.sort(flat[u])[::-1][b - 1]
            assert np.all(np.abs(flat[u][diff] - t) <= 2 * ATOL)
    return same / max(total, 1)


@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_keydiff_whole_path_by_flag(oracle, dtype):
    """lukv_compress with LUKV_FLAG_KEYDIFF: KeyDiff scores -> joint allocation from the curves -> per-head top-b ->
    gather, against the same chain of oracle functions.  No queries are passed."""
    wl = synth.scaled(synth.CONFIGS["llama8b_1layer_8k"], S=2, L=2, H=3, T=4096, w=1, kp=1, P=129, dtype=dtype,
                      d=128 if dtype == "bf16" else 64)
    _, k, v = synth.gen_tensors(wl, "cpu")
    curves = synth.gen_curves(wl)
    n = wl.T - wl.w
    Bs = [int(0.2 * wl.N * n), int(0.55 * wl.N * n)]
    p = lukv.make_params(wl.S, wl.L, wl.H, wl.G, wl.d, wl.T, wl.w, wl.kp, wl.dtype, wl.P, flags=lukv.FLAG_KEYDIFF)
    ws = lukv.alloc_workspace(p)
    out = lukv.Outputs(p, Bs)
    kc, vc = k.cuda(), v.cuda()
    lukv.lukv_compress(p, None, kc, vc, torch.from_numpy(curves).cuda(), Bs, out.k_out, out.v_out, out.kept_idx,
                       out.budgets, out.offsets, out.rows, out.dev_status, ws)
    torch.cuda.synchronize()
    assert int(out.dev_status.item()) == 0
    ref_scores = oracle.keydiff(bits(k), wl.w)
    rb, ro = oracle.allocate(curves, wl.T, wl.w, Bs)
    np.testing.assert_array_equal(out.budgets.cpu().numpy(), rb)
    np.testing.assert_array_equal(out.offsets.cpu().numpy(), ro)
    U = wl.S * wl.N
    rk, rv, rkept = oracle.select_gather(ref_scores.reshape(U, n), rb, ro, bits(k).reshape(U, wl.T, wl.d),
                                         bits(v).reshape(U, wl.T, wl.d), wl.w)
    kept = out.kept_idx.cpu().numpy()
    assert _kept_close(kept, rkept, rb, ro, ref_scores, wl.w) >= 0.999
    # the gathered rows are the rows the kept indices name, bit for bit
    kb, vb = bits(k).reshape(U, wl.T, wl.d), bits(v).reshape(U, wl.T, wl.d)
    head_of_row = np.repeat(np.arange(U), np.diff(ro))
    np.testing.assert_array_equal(bits(out.k_out), kb[head_of_row, kept])
    np.testing.assert_array_equal(bits(out.v_out), vb[head_of_row, kept])
    # lukv_score with the flag returns the KeyDiff scores
    scores = torch.empty((wl.S, wl.N, n), dtype=torch.float32, device="cuda")
    lukv.lukv_score(p, None, kc, scores, ws)
    torch.cuda.synchronize()
    np.testing.assert_allclose(scores.cpu().numpy(), ref_scores, rtol=0, atol=ATOL)


def test_keydiff_flag_in_the_profiling_call():
    """lukv_compress_profile with the flag runs the same kernels one after the other: same bytes, and the timeline
    names the KeyDiff kernel instead of the attention scorer and the pooling."""
    wl = synth.scaled(synth.CONFIGS["llama8b_1layer_8k"], H=3, T=2048, w=1, kp=1, P=65)
    _, k, v = synth.gen_tensors(wl, "cuda")
    curves = torch.from_numpy(synth.gen_curves(wl)).cuda()
    Bs = [int(0.3 * wl.N * (wl.T - 1))]
    p = lukv.make_params(wl.S, wl.L, wl.H, wl.G, wl.d, wl.T, wl.w, wl.kp, wl.dtype, wl.P, flags=lukv.FLAG_KEYDIFF)
    ws = lukv.alloc_workspace(p)
    a, b = lukv.Outputs(p, Bs), lukv.Outputs(p, Bs)
    lukv.lukv_compress(p, None, k, v, curves, Bs, a.k_out, a.v_out, a.kept_idx, a.budgets, a.offsets, a.rows,
                       a.dev_status, ws)
    times = lukv.lukv_compress_profile(p, None, k, v, curves, Bs, b.k_out, b.v_out, b.kept_idx, b.budgets, b.offsets,
                                       b.rows, b.dev_status, ws)
    torch.cuda.synchronize()
    names = [name for name, _ in times]
    assert "keydiff" in names and not any("score" in name or "pool" in name for name in names)
    assert all(ms >= 0.0 for _, ms in times)
    assert torch.equal(a.kept_idx, b.kept_idx) and torch.equal(a.budgets, b.budgets)
    assert torch.equal(a.k_out.view(torch.int16), b.k_out.view(torch.int16))


def test_keydiff_flag_argument_errors():
    f = torch.empty(4096, dtype=torch.uint8, device="cuda")
    pooled = lukv.make_params(1, 1, 2, 1, 64, 256, 1, 7, "bf16", 2, flags=lukv.FLAG_KEYDIFF)   # the metric is not pooled
    assert lukv.lukv_score(pooled, None, f, f, f, check=False) == lukv.ERR_INVALID_ARG
    unknown = lukv.make_params(1, 1, 2, 1, 64, 256, 1, 1, "bf16", 2, flags=2)
    assert lukv.lukv_score(unknown, None, f, f, f, check=False) == lukv.ERR_INVALID_ARG
    plain = lukv.make_params(1, 1, 2, 1, 64, 256, 1, 1, "bf16", 2)
    assert lukv.lukv_score(plain, None, f, f, f, check=False) == lukv.ERR_INVALID_ARG           # queries are required
    flagged = lukv.make_params(2, 1, 2, 1, 64, 256, 1, 1, "bf16", 2, flags=lukv.FLAG_KEYDIFF)
    assert lukv.lukv_score_ragged(flagged, [256, 128], None, f, f, f, check=False) == lukv.ERR_UNSUPPORTED
