"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle, element by element.

Bars: scores within max relative error 2e-3 (+1e-30 absolute at the underflow edge);
allocation, selection and gather bit-exact when run on the oracle's own curves and scores;
end-to-end kept-index agreement >= 99.9 % with every mismatch at a score gap below the
tolerance.
"""
import numpy as np
import pytest
import torch

from paper_2602_08585_b200 import lukv, synth
from gpu_helpers import (assert_scores_close, bits, gpu_allocate, gpu_compress, gpu_score, gpu_select_gather,
                         kept_agreement, params_of)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _need_gpu():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    lukv.lib()


def _rand_qkv(S, L, H, G, d, T, w, dtype, seed, scale=1.0):
    g = torch.Generator(device="cpu").manual_seed(seed)
    q = (torch.randn((S, L, H * G, w, d), generator=g) * scale).to(dtype)
    k = (torch.randn((S, L, H, T, d), generator=g) * scale).to(dtype)
    v = torch.randn((S, L, H, T, d), generator=g).to(dtype)
    return q, k, v


# ---- stage (a): scores -------------------------------------------------------------------------

SCORE_SHAPES = [
    # S, L, H, G, d,   T,   w, kp, dtype
    (1, 1, 1, 1, 64, 2, 1, 1, torch.float32),          # smallest legal problem
    (1, 1, 2, 1, 64, 77, 5, 3, torch.float32),         # ragged everything
    (2, 1, 2, 3, 64, 1025, 7, 5, torch.bfloat16),      # one key past a chunk
    (1, 2, 1, 4, 128, 1300, 32, 7, torch.bfloat16),    # 128 rows, ragged tail
    (1, 1, 1, 7, 128, 2048, 32, 7, torch.bfloat16),    # 224 rows (GQA group 7)
    (1, 1, 1, 4, 128, 1111, 64, 5, torch.bfloat16),    # 256 rows
    (1, 1, 2, 2, 128, 640, 16, 9, torch.float32),
    (1, 1, 1, 1, 128, 4096 + 33, 33, 1, torch.bfloat16),
]


@pytest.mark.parametrize("shape", SCORE_SHAPES)
def test_score_matches_oracle(oracle, shape):
    S, L, H, G, d, T, w, kp, dtype = shape
    q, k, _ = _rand_qkv(S, L, H, G, d, T, w, dtype, seed=T + w, scale=2.0)
    p = lukv.make_params(S, L, H, G, d, T, w, kp, dtype, 2)
    got = gpu_score(p, q.cuda(), k.cuda()).cpu().numpy()
    ref = oracle.score(bits(q), bits(k), G, kp)
    assert_scores_close(got, ref)


def test_score_explicit_scale(oracle):
    S, L, H, G, d, T, w, kp = 1, 1, 2, 2, 64, 300, 4, 3
    q, k, _ = _rand_qkv(S, L, H, G, d, T, w, torch.bfloat16, seed=5)
    p = lukv.make_params(S, L, H, G, d, T, w, kp, torch.bfloat16, 2, scale=0.3)
    got = gpu_score(p, q.cuda(), k.cuda()).cpu().numpy()
    assert_scores_close(got, oracle.score(bits(q), bits(k), G, kp, scale=0.3))


@pytest.mark.parametrize("name", ["tiny", "llama8b_1layer_8k"])
def test_score_on_benchmark_configs(oracle, name):
    wl = synth.CONFIGS[name]
    q, k, _ = synth.gen_tensors(wl, "cuda")
    qc, kc, _ = synth.gen_tensors(wl, "cpu")
    assert torch.equal(q.cpu(), qc) and torch.equal(k.cpu(), kc)      # same bits on both devices
    got = gpu_score(params_of(wl), q, k).cpu().numpy()
    ref = oracle.score(bits(qc), bits(kc), wl.G, wl.kp)
    assert_scores_close(got, ref)


# ---- stage (b): allocation ---------------------------------------------------------------------

def _alloc_case(oracle, N, P, T, w, curves, Bs, L=None):
    L = L or 1
    p = lukv.make_params(len(Bs), L, N // L, 1, 64, T, w, 1, torch.bfloat16, P)
    b_gpu, o_gpu = gpu_allocate(p, curves, Bs)
    b_ref, o_ref = oracle.allocate(curves, T, w, Bs)
    np.testing.assert_array_equal(b_gpu, b_ref)
    np.testing.assert_array_equal(o_gpu, o_ref)


@pytest.mark.parametrize("name", list(synth.CONFIGS))
def test_allocate_bit_exact_on_benchmark_configs(oracle, name):
    wl = synth.CONFIGS[name]
    curves = synth.gen_curves(wl)
    p = params_of(wl)
    b_gpu, o_gpu = gpu_allocate(p, curves, wl.budgets())
    b_ref, o_ref = oracle.allocate(curves, wl.T, wl.w, wl.budgets())
    np.testing.assert_array_equal(b_gpu, b_ref)
    np.testing.assert_array_equal(o_gpu, o_ref)
    np.testing.assert_array_equal(b_gpu.sum(axis=1), wl.budgets())
    assert o_gpu[-1] == wl.total_rows()


def test_allocate_edge_cases(oracle):
    rng = np.random.default_rng(0)
    N, P, T, w = 12, 9, 64, 5          # s = 8, n = 59: last segment holds 3 tokens
    inc = rng.exponential(size=(N, P - 1))
    U = np.zeros((N, P), np.float32)
    U[:, 1:] = np.cumsum(inc, axis=1)
    n = T - w
    _alloc_case(oracle, N, P, T, w, U, [0, 1, 100, 333, N * n - 1, N * n])
    # flat and identical curves: every gain ties, order falls back to (k, hid)
    flat = np.tile(np.arange(P, dtype=np.float32), (N, 1))
    _alloc_case(oracle, N, P, T, w, flat, [7, 8 * N + 3, 50 * N + 1, N * n])
    # concave, integer valued (exact ties between heads), decreasing tails (zero gains)
    conc = np.zeros((N, P), np.float32)
    conc[:, 1:] = np.cumsum(np.arange(P - 1, 0, -1, dtype=np.float64))[None, :]
    _alloc_case(oracle, N, P, T, w, conc, [N * 8 * 3, 100, 401])
    dip = U.copy()
    dip[:, 5:] -= np.arange(1, P - 4, dtype=np.float32)[None, :] * 3.0
    _alloc_case(oracle, N, P, T, w, dip, [50, 300, N * n])
    # window wider than a segment: several trailing segments are unusable
    _alloc_case(oracle, N, 17, 64, 21, np.ascontiguousarray(np.repeat(U, 2, axis=1)[:, :17]), [10, 200, N * 43])
    # all-zero curves (every gain is +0)
    _alloc_case(oracle, N, P, T, w, np.zeros((N, P), np.float32), [0, 77, N * n])


def test_allocate_many_sequences_and_many_heads(oracle):
    rng = np.random.default_rng(1)
    N, P, T, w = 300, 33, 1024, 16     # more heads than threads of one allocation CTA
    inc = rng.exponential(size=(N, P - 1)) * np.where(rng.random((N, P - 1)) < 0.2, 3.0, 1.0)
    U = np.zeros((N, P), np.float32)
    U[:, 1:] = np.cumsum(inc, axis=1)
    Bs = [int(x) for x in rng.integers(0, N * (T - w), size=40)]     # more sequences than one launch takes
    _alloc_case(oracle, N, P, T, w, U, Bs, L=3)


def test_allocate_long_curves(oracle):
    rng = np.random.default_rng(2)
    N, P, T, w = 5, 4097, 4096, 32
    inc = rng.exponential(size=(N, P - 1)) * np.where(rng.random((N, P - 1)) < 0.2, 3.0, 1.0)
    U = np.zeros((N, P), np.float32)
    U[:, 1:] = np.cumsum(inc, axis=1)
    _alloc_case(oracle, N, P, T, w, U, [1234, 9999])


# ---- stages (c)+(d): selection and gather on the oracle's scores ------------------------------------

def _select_case(oracle, S, N, T, w, d, dtype, budgets, scores, seed=0):
    g = torch.Generator().manual_seed(seed)
    k = torch.randn((S, 1, N, T, d), generator=g).to(dtype)
    v = torch.randn((S, 1, N, T, d), generator=g).to(dtype)
    budgets = np.asarray(budgets, np.int32).reshape(S, N)
    offsets = np.concatenate([[0], np.cumsum(budgets.reshape(-1) + w)]).astype(np.int32)
    rows = int(offsets[-1])
    p = lukv.make_params(S, 1, N, 1, d, T, w, 1, dtype, 2)
    k_out, v_out, kept = gpu_select_gather(p, torch.from_numpy(scores).cuda(), torch.from_numpy(budgets).cuda(),
                                           torch.from_numpy(offsets).cuda(), k.cuda(), v.cuda(), rows, pad_rows=3)
    rk, rv, rkept = oracle.select_gather(scores.reshape(S * N, T - w), budgets, offsets, bits(k).reshape(S * N, T, d),
                                         bits(v).reshape(S * N, T, d), w)
    np.testing.assert_array_equal(kept.cpu().numpy()[:rows], rkept)
    np.testing.assert_array_equal(bits(k_out)[:rows], rk)
    np.testing.assert_array_equal(bits(v_out)[:rows], rv)
    # rows beyond rows_cap are never written
    assert torch.all(kept[rows:] == -1) and torch.all(k_out[rows:] == 0) and torch.all(v_out[rows:] == 0)


@pytest.mark.parametrize("T,w,d,dtype", [(77, 5, 64, torch.float32), (1024, 16, 64, torch.float32),
                                         (5000, 32, 128, torch.bfloat16), (20000, 32, 128, torch.bfloat16),
                                         (33000, 64, 64, torch.bfloat16), (40000, 32, 128, torch.float32)])
def test_select_gather_bit_exact(oracle, T, w, d, dtype):
    rng = np.random.default_rng(T)
    S, N, n = 2, 3, T - w
    scores = rng.random((S, N, n)).astype(np.float32) ** 8
    scores[0, 1] = np.repeat(rng.random(n // 7 + 1).astype(np.float32), 7)[:n]     # plateaus: ties at the cut
    scores[1, 0] = 0.0                                                               # all equal
    scores[1, 2, ::3] = 0.0
    budgets = [0, n // 3, n, 17 % n, 1, n - 1]
    _select_case(oracle, S, N, T, w, d, dtype, budgets, scores, seed=T)


def test_select_gather_long_context_single_head(oracle):
    T, w, d = 131072, 32, 128
    rng = np.random.default_rng(9)
    scores = np.maximum(rng.standard_normal((1, 1, T - w)).astype(np.float32), 0.0)   # half the scores tie at 0
    _select_case(oracle, 1, 1, T, w, d, torch.bfloat16, [90000], scores)


@pytest.mark.parametrize("T,n_sink", [(70000, 0), (131072 + 64, 4), (200000, 0), (262144 + 32, 0), (270000, 4)])
def test_select_gather_cluster_and_streaming_paths(oracle, T, n_sink):
    """Contexts beyond 32768 positions: clusters of 4 and 8 CTAs per head that merge their histograms (clusters of 2:
    the 33000 and 40000 cases above), and beyond 262144 positions one CTA that re-reads its keys.  Plateaus put ties
    on the cut; one head keeps nothing, one nearly everything."""
    w, d, S, N = 32, 64, 1, 3
    n = T - w
    rng = np.random.default_rng(T)
    scores = rng.random((S, N, n)).astype(np.float32) ** 8
    scores[0, 1] = np.repeat(rng.random(n // 5 + 1).astype(np.float32), 5)[:n]
    budgets = np.asarray([[n // 3, n - 7, 0]], np.int32)
    if n_sink:
        scores[0, 0, :n_sink] = 0.0                    # sinks rank first whatever their scores
    g = torch.Generator().manual_seed(T)
    k = torch.randn((S, 1, N, T, d), generator=g).to(torch.bfloat16)
    v = torch.randn((S, 1, N, T, d), generator=g).to(torch.bfloat16)
    offsets = np.concatenate([[0], np.cumsum(budgets.reshape(-1) + w)]).astype(np.int32)
    rows = int(offsets[-1])
    p = lukv.make_params(S, 1, N, 1, d, T, w, 1, torch.bfloat16, 2, n_sink=n_sink)
    k_out, v_out, kept = gpu_select_gather(p, torch.from_numpy(scores).cuda(), torch.from_numpy(budgets).cuda(),
                                           torch.from_numpy(offsets).cuda(), k.cuda(), v.cuda(), rows, pad_rows=3)
    rk, rv, rkept = oracle.select_gather(scores.reshape(N, n), budgets, offsets, bits(k).reshape(N, T, d),
                                         bits(v).reshape(N, T, d), w, n_sink=n_sink)
    np.testing.assert_array_equal(kept.cpu().numpy()[:rows], rkept)
    np.testing.assert_array_equal(bits(k_out)[:rows], rk)
    np.testing.assert_array_equal(bits(v_out)[:rows], rv)
    assert torch.all(kept[rows:] == -1)


# ---- the whole path ------------------------------------------------------------------------------

def _compress_case(oracle, wl, min_agreement=0.999):
    q, k, v = synth.gen_tensors(wl, "cuda")
    curves = synth.gen_curves(wl)
    Bs = wl.budgets()
    out = gpu_compress(params_of(wl), q, k, v, curves, Bs)
    ref = oracle.compress(bits(q), bits(k), bits(v), curves, Bs, wl.G, wl.kp)
    budgets = out.budgets.cpu().numpy()
    offsets = out.offsets.cpu().numpy()
    kept = out.kept_idx.cpu().numpy()
    np.testing.assert_array_equal(budgets, ref["budgets"])
    np.testing.assert_array_equal(offsets, ref["offsets"])
    agree = kept_agreement(kept, ref["kept_idx"], offsets, budgets, ref["scores"])
    assert agree >= min_agreement, f"kept-index agreement {agree:.5f}"
    # packed rows are bit-exact copies of the rows kept_idx names (window rows included)
    kb, vb = bits(k).reshape(wl.S * wl.N, wl.T, wl.d), bits(v).reshape(wl.S * wl.N, wl.T, wl.d)
    ko, vo = bits(out.k_out), bits(out.v_out)
    for u in range(wl.S * wl.N):
        lo, hi = offsets[u], offsets[u + 1]
        np.testing.assert_array_equal(ko[lo:hi], kb[u][kept[lo:hi]])
        np.testing.assert_array_equal(vo[lo:hi], vb[u][kept[lo:hi]])
        np.testing.assert_array_equal(kept[hi - wl.w:hi], np.arange(wl.n, wl.T))
    # identical index sets => identical packed bytes
    same = kept == ref["kept_idx"]
    np.testing.assert_array_equal(ko[same], ref["k_out"][same])
    np.testing.assert_array_equal(vo[same], ref["v_out"][same])
    return agree


@pytest.mark.parametrize("name", ["tiny", "llama8b_1layer_8k"])
def test_compress_on_benchmark_configs(oracle, name):
    _compress_case(oracle, synth.CONFIGS[name])


def test_compress_reduced_batch_mixed_budgets(oracle):
    # the batched mixed-budget configuration at reduced size: 2 layers x 2 heads, 4 sequences
    wl = synth.scaled(synth.CONFIGS["batch8_16k_mixed"], S=4, L=2, H=2, T=2048, P=33, needles=16)
    _compress_case(oracle, wl)


def test_compress_reduced_gqa7_student_t(oracle):
    wl = synth.scaled(synth.CONFIGS["gqa7_128k"], L=1, H=2, T=4096, P=65, needles=32)
    _compress_case(oracle, wl)


def test_compress_is_deterministic():
    wl = synth.scaled(synth.CONFIGS["llama8b_1layer_8k"], H=2, T=4096, P=65)
    q, k, v = synth.gen_tensors(wl, "cuda")
    curves = synth.gen_curves(wl)
    a = gpu_compress(params_of(wl), q, k, v, curves, wl.budgets())
    b = gpu_compress(params_of(wl), q, k, v, curves, wl.budgets())
    assert torch.equal(a.kept_idx, b.kept_idx) and torch.equal(a.k_out.view(torch.int16), b.k_out.view(torch.int16))
    assert torch.equal(a.budgets, b.budgets) and torch.equal(a.offsets, b.offsets)


@pytest.mark.parametrize("kw", [
    dict(L=2, H=4, T=8192, P=129),                         # 128 query rows per head: one row block
    dict(L=1, H=3, G=7, T=6000 + 96, w=32, P=2),           # 224 query rows: two row blocks, ragged last key tile
    dict(S=3, L=1, H=5, T=3000 + 40, w=40, kp=5, P=2),     # 160 rows, several sequences, short items
    dict(L=1, H=40, T=1024, P=2),                          # fewer work items than CTAs per head
])
def test_tensor_core_scorer_repeats_bit_for_bit(kw):
    """The persistent scorer's CTAs hand partial results to one another; a rare ordering bug there shows as a
    repetition whose bits differ.  Every reduction has a fixed order, so 40 repetitions must be identical."""
    wl = synth.scaled(synth.CONFIGS["llama8b_1layer_8k"], needles=16, **kw)
    p = params_of(wl)
    q, k, _ = synth.gen_tensors(wl, "cuda")
    ws = lukv.alloc_workspace(p)
    first = torch.empty((p.batch, p.N, p.n), dtype=torch.float32, device="cuda")
    lukv.lukv_score(p, q, k, first, ws)
    again = torch.empty_like(first)
    for rep in range(40):
        again.fill_(-1.0)
        lukv.lukv_score(p, q, k, again, ws)
        assert torch.equal(again, first), rep
    assert torch.isfinite(first).all() and (first >= 0).all()


def test_allocate_more_heads_than_threads(oracle):
    # 1500 heads: the allocation CTA (at most 1024 threads, one head each) loops over the heads
    rng = np.random.default_rng(9)
    N, P, T, w = 1500, 17, 256, 16
    inc = rng.exponential(size=(N, P - 1)) * np.where(rng.random((N, P - 1)) < 0.2, 3.0, 1.0)
    U = np.zeros((N, P), np.float32)
    U[:, 1:] = np.cumsum(inc, axis=1)
    U[::7] = U[3]                        # many identical heads: ties across heads
    n = T - w
    _alloc_case(oracle, N, P, T, w, U, [0, 1, 12345, N * n // 3, N * n - 1, N * n], L=3)


def test_three_quad_scorer_variant_in_a_subprocess(oracle):
    """LUKV_QUADS=3 selects the scorer with three epilogue quads (read once per process, hence the
    subprocess); it must meet the same tolerance and repeat bit for bit."""
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    code = f"""
import sys
sys.path.insert(0, {root!r}); sys.path.insert(0, {os.path.join(root, 'tests')!r})
import numpy as np, torch
from paper_2602_08585_b200 import lukv, synth
from oracle import lukv_oracle
from gpu_helpers import params_of, gpu_score, assert_scores_close, bits
wl = synth.scaled(synth.CONFIGS["llama8b_1layer_8k"], L=2, H=3, T=6000 + 32, P=2, needles=16)
q, k, _ = synth.gen_tensors(wl, "cuda")
p = params_of(wl)
a = gpu_score(p, q, k)
b = gpu_score(p, q, k)
assert torch.equal(a, b)
ref = lukv_oracle.score(bits(q), bits(k), wl.G, wl.kp)
assert_scores_close(a.cpu().numpy(), ref)
print("ok")
"""
    env = dict(os.environ, LUKV_QUADS="3")
    out = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0 and "ok" in out.stdout, out.stderr[-2000:]


def test_compress_can_be_captured_in_a_cuda_graph():
    """The whole call only enqueues (kernels, two small memsets, an event pair on the auxiliary stream), so a caller
    may capture it into a CUDA graph; replays give the same bytes as the plain call."""
    wl = synth.scaled(synth.CONFIGS["llama8b_1layer_8k"], H=4, T=4096, P=65)
    q, k, v = synth.gen_tensors(wl, "cuda")
    curves = torch.from_numpy(synth.gen_curves(wl)).cuda()
    Bs = wl.budgets()
    p = params_of(wl)
    ws = lukv.alloc_workspace(p)
    plain, out = lukv.Outputs(p, Bs), lukv.Outputs(p, Bs)

    def call(o):
        lukv.lukv_compress(p, q, k, v, curves, Bs, o.k_out, o.v_out, o.kept_idx, o.budgets, o.offsets, o.rows,
                           o.dev_status, ws)

    call(plain)
    torch.cuda.synchronize()
    graph, side = torch.cuda.CUDAGraph(), torch.cuda.Stream()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            call(out)
    for _ in range(3):
        out.kept_idx.fill_(-1)
        out.k_out.zero_()
        graph.replay()
    torch.cuda.synchronize()
    assert int(out.dev_status.item()) == 0
    assert torch.equal(out.budgets, plain.budgets) and torch.equal(out.kept_idx, plain.kept_idx)
    assert torch.equal(out.k_out.view(torch.int16), plain.k_out.view(torch.int16))
    assert torch.equal(out.v_out.view(torch.int16), plain.v_out.view(torch.int16))
