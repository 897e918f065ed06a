"""GPU parity of the deployment settings of App. E (attention sinks, minimum retention per head) and of
layer-by-layer use of the entry points, against the oracle."""
import numpy as np
import pytest
import torch

from paper_2602_08585_b200 import lukv, synth
from gpu_helpers import bits, gpu_allocate, gpu_compress, gpu_select_gather, kept_agreement

pytestmark = pytest.mark.gpu


def _params(wl, **kw):
    return lukv.make_params(wl.S, wl.L, wl.H, wl.G, wl.d, wl.T, wl.w, wl.kp, wl.dtype, wl.P, **kw)


def _rough(rng, N, P):
    inc = rng.exponential(size=(N, P - 1)) * np.where(rng.random((N, P - 1)) < 0.2, 3.0, 1.0)
    U = np.zeros((N, P), np.float32)
    U[:, 1:] = np.cumsum(inc, axis=1)
    return U


@pytest.mark.parametrize("name", list(synth.CONFIGS))
def test_allocate_with_floor_on_benchmark_configs(oracle, name):
    wl = synth.CONFIGS[name]
    curves = synth.gen_curves(wl)
    curves[1::5] *= 1e-4                  # heads the plain greedy would starve
    b_gpu, o_gpu = gpu_allocate(_params(wl, min_keep=0.01), curves, wl.budgets())
    b_ref, o_ref = oracle.allocate(curves, wl.T, wl.w, wl.budgets(), min_keep=0.01)
    np.testing.assert_array_equal(b_gpu, b_ref)
    np.testing.assert_array_equal(o_gpu, o_ref)
    f = oracle.floor_tokens(0.01, wl.n)
    assert b_gpu.min() == f
    np.testing.assert_array_equal(b_gpu.sum(axis=1), wl.budgets())


def test_allocate_with_floor_edge_cases(oracle):
    rng = np.random.default_rng(40)
    N, P, T, w = 12, 9, 64, 5             # s = 8, n = 59
    n = T - w
    U = _rough(rng, N, P)
    U[4] = 0.0
    for mk in (0.03, 0.125, 0.2, 0.5, 1.0):   # floors of 2, 8 (a whole segment), 12, 30 and n tokens
        f = oracle.floor_tokens(mk, n)
        Bs = sorted({N * f, min(N * f + 1, N * n), (N * f + N * n) // 2, N * n - 1 if N * n - 1 >= N * f else N * n,
                     N * n})
        p = lukv.make_params(len(Bs), 1, N, 1, 64, T, w, 1, torch.bfloat16, P, min_keep=mk)
        b_gpu, o_gpu = gpu_allocate(p, U, Bs)
        b_ref, o_ref = oracle.allocate(U, T, w, Bs, min_keep=mk)
        np.testing.assert_array_equal(b_gpu, b_ref)
        np.testing.assert_array_equal(o_gpu, o_ref)
        assert b_gpu.min() >= f
    # token-resolution curves, more sequences than one launch takes
    N, T, w = 20, 256, 16
    U = _rough(rng, N, T + 1)
    n = T - w
    f = oracle.floor_tokens(0.05, n)
    Bs = [int(x) for x in rng.integers(N * f, N * n, size=40)]
    p = lukv.make_params(len(Bs), 2, N // 2, 1, 64, T, w, 1, torch.bfloat16, T + 1, min_keep=0.05)
    b_gpu, o_gpu = gpu_allocate(p, U, Bs)
    b_ref, o_ref = oracle.allocate(U, T, w, Bs, min_keep=0.05)
    np.testing.assert_array_equal(b_gpu, b_ref)
    np.testing.assert_array_equal(o_gpu, o_ref)


@pytest.mark.parametrize("T,w", [(300, 7), (1500, 32), (8192, 32), (40000, 32)])   # all four register layouts
def test_select_with_sinks(oracle, T, w):
    rng = np.random.default_rng(T)
    S, N, d, n = 1, 3, 64, T - w
    scores = rng.random((S * N, n)).astype(np.float32)
    scores[:, :4] = 0.0                   # the sinks score lowest: only the setting keeps them
    scores[1, 100:130] = scores[1, 100]   # ties
    budgets = np.array([[2, n // 5, n]], np.int32)
    offsets = np.concatenate([[0], np.cumsum(budgets.reshape(-1) + w)]).astype(np.int32)
    rows = int(offsets[-1])
    g = torch.Generator().manual_seed(1)
    k = torch.randn((S, 1, N, T, d), generator=g).to(torch.bfloat16)
    v = torch.randn((S, 1, N, T, d), generator=g).to(torch.bfloat16)
    p = lukv.make_params(S, 1, N, 1, d, T, w, 1, torch.bfloat16, 2, n_sink=4)
    k_out, v_out, kept = gpu_select_gather(p, torch.from_numpy(scores).cuda(), torch.from_numpy(budgets).cuda(),
                                           torch.from_numpy(offsets).cuda(), k.cuda(), v.cuda(), rows)
    k_ref, v_ref, kept_ref = oracle.select_gather(scores, budgets, offsets, bits(k), bits(v), w, n_sink=4)
    np.testing.assert_array_equal(kept.cpu().numpy(), kept_ref)
    np.testing.assert_array_equal(bits(k_out), k_ref)
    np.testing.assert_array_equal(bits(v_out), v_ref)
    kept = kept.cpu().numpy()
    assert list(kept[:2]) == [0, 1]                                   # budget below the sink count
    assert list(kept[offsets[1]:offsets[1] + 4]) == [0, 1, 2, 3]


@pytest.mark.parametrize("name", ["tiny", "llama8b_1layer_8k"])
def test_compress_with_sinks_and_floor(oracle, name):
    wl = synth.CONFIGS[name]
    q, k, v = synth.gen_tensors(wl, "cuda")
    curves = synth.gen_curves(wl)
    curves[1] *= 1e-4
    Bs = wl.budgets()
    out = gpu_compress(_params(wl, n_sink=4, min_keep=0.01), q, k, v, curves, Bs)
    ref = oracle.compress(bits(q), bits(k), bits(v), curves, Bs, wl.G, wl.kp, n_sink=4, min_keep=0.01)
    budgets, offsets, kept = out.budgets.cpu().numpy(), out.offsets.cpu().numpy(), out.kept_idx.cpu().numpy()
    np.testing.assert_array_equal(budgets, ref["budgets"])
    np.testing.assert_array_equal(offsets, ref["offsets"])
    assert budgets.min() == oracle.floor_tokens(0.01, wl.n)
    assert kept_agreement(kept, ref["kept_idx"], offsets, budgets, ref["scores"], n_sink=4) >= 0.999
    kb, vb = bits(k).reshape(wl.S * wl.N, wl.T, wl.d), bits(v).reshape(wl.S * wl.N, wl.T, wl.d)
    ko, vo = bits(out.k_out), bits(out.v_out)
    for u in range(wl.S * wl.N):
        lo, hi = offsets[u], offsets[u + 1]
        assert list(kept[lo:lo + 4]) == [0, 1, 2, 3]
        np.testing.assert_array_equal(ko[lo:hi], kb[u][kept[lo:hi]])
        np.testing.assert_array_equal(vo[lo:hi], vb[u][kept[lo:hi]])


def test_profile_path_with_floor(oracle):
    L, H, T, w, Mq = 2, 6, 256, 16, 4
    U = synth.gen_calibration_curves(303, Mq, L * H, T)
    ratios = np.linspace(0.0, 1.0, 41).astype(np.float32)
    calib = lukv.make_params(1, L, H, 1, 64, T, w, 1, "fp32", T + 1, min_keep=0.02)
    ws = torch.empty(lukv.lukv_profile_workspace_bytes(calib, Mq, len(ratios)), dtype=torch.uint8, device="cuda")
    phi = torch.empty((len(ratios), L * H), dtype=torch.float32, device="cuda")
    lukv.lukv_profile_build(calib, torch.from_numpy(U).cuda(), Mq, ratios, phi, ws)
    torch.cuda.synchronize()
    ref = oracle.profile_build(U, T, w, ratios, min_keep=0.02)
    np.testing.assert_array_equal(phi.cpu().numpy(), ref)
    assert ref.max() < 1.0
    S, Tn = 5, 5000
    sigma = np.array([0.0, 0.5, 0.9, 0.99, 1.0], np.float32)
    p = lukv.make_params(S, L, H, 4, 128, Tn, 32, 7, "bf16", 3, min_keep=0.02)
    budgets = torch.empty((S, L * H), dtype=torch.int32, device="cuda")
    offsets = torch.empty((S * L * H + 1,), dtype=torch.int32, device="cuda")
    lukv.lukv_profile_budgets(p, phi, ratios, sigma, budgets, offsets)
    torch.cuda.synchronize()
    b_ref, o_ref = oracle.profile_budgets(ref, ratios, Tn, 32, sigma, min_keep=0.02)
    np.testing.assert_array_equal(budgets.cpu().numpy(), b_ref)
    np.testing.assert_array_equal(offsets.cpu().numpy(), o_ref)
    assert b_ref.min() >= oracle.floor_tokens(0.02, Tn - 32)


def test_layer_by_layer_equals_one_call(oracle):
    """A server can compress layer l as soon as its prefill is done: allocation once for the whole model
    (it only needs the curves), then scoring, selection and gather with one-layer parameters on that layer's
    tensors and its slice of the budgets and offsets.  The packed cache is the same as from one call."""
    wl = synth.scaled(synth.CONFIGS["llama8b_1layer_8k"], L=3, H=2, T=4096, P=65)
    q, k, v = synth.gen_tensors(wl, "cuda")
    curves = synth.gen_curves(wl)
    Bs = wl.budgets()
    whole = gpu_compress(_params(wl, n_sink=4), q, k, v, curves, Bs)
    p_all = _params(wl, n_sink=4)
    ws = lukv.alloc_workspace(p_all)
    budgets = torch.empty((1, wl.N), dtype=torch.int32, device="cuda")
    offsets = torch.empty((wl.N + 1,), dtype=torch.int32, device="cuda")
    lukv.lukv_allocate(p_all, torch.from_numpy(curves).cuda(), Bs, budgets, offsets, ws)
    rows = whole.rows
    k_out = torch.zeros((rows, wl.d), dtype=k.dtype, device="cuda")
    v_out = torch.zeros((rows, wl.d), dtype=k.dtype, device="cuda")
    kept = torch.full((rows,), -1, dtype=torch.int32, device="cuda")
    p1 = lukv.make_params(1, 1, wl.H, wl.G, wl.d, wl.T, wl.w, wl.kp, wl.dtype, wl.P, n_sink=4)
    ws1 = lukv.alloc_workspace(p1)
    scores = torch.empty((1, wl.H, wl.n), dtype=torch.float32, device="cuda")
    for layer in range(wl.L):
        lukv.lukv_score(p1, q[0, layer], k[0, layer], scores, ws1)
        lukv.lukv_select_gather(p1, scores, budgets[0, layer * wl.H:], offsets[layer * wl.H:], k[0, layer],
                                v[0, layer], k_out, v_out, kept, rows, ws1)
    torch.cuda.synchronize()
    assert torch.equal(budgets, whole.budgets) and torch.equal(offsets, whole.offsets)
    assert torch.equal(kept, whole.kept_idx)
    assert torch.equal(k_out.view(torch.int16), whole.k_out.view(torch.int16))
    assert torch.equal(v_out.view(torch.int16), whole.v_out.view(torch.int16))
