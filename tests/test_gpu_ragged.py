"""GPU parity of a batch whose sequences have different context lengths (one lukv_compress_ragged call)
against the oracle, which by definition runs the sequences one by one.  Budgets and offsets are bit-exact;
scores within the tolerance; kept-index agreement >= 99.9 % with every mismatch at the threshold; packed
rows are exact copies; padding behind a sequence's last position is never used."""
import numpy as np
import pytest
import torch

from paper_2602_08585_b200 import lukv, synth
from gpu_helpers import assert_scores_close, bits, kept_agreement

pytestmark = pytest.mark.gpu


def _case(oracle, S, L, H, G, d, T, w, kp, P, dtype, lens, keep, seed, n_sink=0, min_keep=0.0):
    g = torch.Generator().manual_seed(seed)
    q = (torch.randn((S, L, H * G, w, d), generator=g) * 1.5).to(dtype)
    k = (torch.randn((S, L, H, T, d), generator=g) * 1.5).to(dtype)
    v = torch.randn((S, L, H, T, d), generator=g).to(dtype)
    for s, Ts in enumerate(lens):                      # poison the padding: it must not matter
        k[s, :, :, Ts:] = 50.0
        v[s, :, :, Ts:] = -7.0
    N = L * H
    rng = np.random.default_rng(seed)
    curves = np.zeros((N, P), np.float32)
    curves[:, 1:] = np.cumsum(rng.exponential(size=(N, P - 1)) * np.where(rng.random((N, P - 1)) < 0.2, 3.0, 1.0), axis=1)
    Bs = [int(keep[s % len(keep)] * N * (lens[s] - w)) for s in range(S)]
    p = lukv.make_params(S, L, H, G, d, T, w, kp, dtype, P, n_sink=n_sink, min_keep=min_keep)
    ws = lukv.alloc_workspace(p)
    out = lukv.Outputs(p, Bs)
    qc, kc, vc = q.cuda(), k.cuda(), v.cuda()
    lukv.lukv_compress_ragged(p, lens, qc, kc, vc, torch.from_numpy(curves).cuda(), Bs, out.k_out, out.v_out,
                              out.kept_idx, out.budgets, out.offsets, out.rows, out.dev_status, ws)
    scores = torch.zeros((S, N, T - w), dtype=torch.float32, device="cuda")
    lukv.lukv_score_ragged(p, lens, qc, kc, scores, ws)
    torch.cuda.synchronize()
    assert int(out.dev_status.item()) == 0
    ref = oracle.compress_ragged(bits(q), bits(k), bits(v), curves, Bs, lens, G, kp, n_sink=n_sink, min_keep=min_keep)
    budgets, offsets = out.budgets.cpu().numpy(), out.offsets.cpu().numpy()
    np.testing.assert_array_equal(budgets, ref["budgets"])
    np.testing.assert_array_equal(offsets, ref["offsets"])
    kept = out.kept_idx.cpu().numpy()
    got_scores = scores.cpu().numpy()
    k_bits, v_bits = bits(k), bits(v)
    k_out, v_out = bits(out.k_out), bits(out.v_out)
    agree_num = agree_den = 0
    for s, Ts in enumerate(lens):
        n_s = Ts - w
        assert_scores_close(got_scores[s, :, :n_s], ref["scores"][s])
        sl = slice(s * N, (s + 1) * N)
        r0, r1 = offsets[s * N], offsets[(s + 1) * N]
        a = kept_agreement(kept[r0:r1], ref["kept_idx"][r0:r1], offsets[s * N:(s + 1) * N + 1] - r0, budgets[s],
                           ref["scores"][s], n_sink=n_sink)
        agree_num += a * budgets[s].sum()
        agree_den += budgets[s].sum()
        for hh in range(N):
            u = s * N + hh
            o, b = offsets[u], budgets.reshape(-1)[u]
            np.testing.assert_array_equal(kept[o + b:o + b + w], np.arange(n_s, Ts))       # the sequence's own window
            rows = kept[o:o + b + w]
            assert rows.max() < Ts
            layer, h = divmod(hh, H)
            np.testing.assert_array_equal(k_out[o:o + b + w], k_bits[s, layer, h][rows])
            np.testing.assert_array_equal(v_out[o:o + b + w], v_bits[s, layer, h][rows])
    assert agree_den == 0 or agree_num / agree_den >= 0.999


def test_three_lengths_tensor_core_scorer(oracle):
    # bf16, head_dim 128: the tensor-core scorer deals work items per sequence; 1280 is not a multiple of 128 keys
    # minus window, 2432 = 19 key tiles
    _case(oracle, 3, 2, 2, 4, 128, 4096, 32, 7, 33, torch.bfloat16, [4096, 1280, 2432], [0.2, 0.5], seed=1)


def test_two_row_blocks_and_sinks(oracle):
    _case(oracle, 2, 1, 2, 4, 128, 2048, 64, 5, 17, torch.bfloat16, [1024, 2048], [0.3], seed=2, n_sink=4, min_keep=0.05)


def test_general_shape_scorer(oracle):
    # fp32, head_dim 64: the FP32-pipe scorer; lengths down to barely more than the window
    _case(oracle, 4, 1, 3, 2, 64, 640, 8, 3, 9, torch.float32, [640, 16, 328, 64], [0.25, 0.6], seed=3)


def test_equal_lengths_match_the_batched_call():
    wl = synth.scaled(synth.CONFIGS["llama8b_1layer_8k"], S=2, H=2, T=2048, P=33, needles=16)
    p = lukv.make_params(wl.S, wl.L, wl.H, wl.G, wl.d, wl.T, wl.w, wl.kp, wl.dtype, wl.P)
    q, k, v = synth.gen_tensors(wl, "cuda")
    curves = torch.from_numpy(synth.gen_curves(wl)).cuda()
    Bs = wl.budgets()
    ws = lukv.alloc_workspace(p)
    a, b = lukv.Outputs(p, Bs), lukv.Outputs(p, Bs)
    lukv.lukv_compress(p, q, k, v, curves, Bs, a.k_out, a.v_out, a.kept_idx, a.budgets, a.offsets, a.rows, a.dev_status, ws)
    lukv.lukv_compress_ragged(p, [wl.T] * wl.S, q, k, v, curves, Bs, b.k_out, b.v_out, b.kept_idx, b.budgets, b.offsets,
                              b.rows, b.dev_status, ws)
    torch.cuda.synchronize()
    assert torch.equal(a.budgets, b.budgets) and torch.equal(a.offsets, b.offsets)
    assert torch.equal(a.kept_idx, b.kept_idx)
    assert torch.equal(a.k_out.view(torch.int16), b.k_out.view(torch.int16))


def test_online_mode_on_sequences_of_different_lengths(oracle):
    """The deployment mode of Sec. 4.3 (lookup and budgeting -> scoring -> eviction) on a ragged batch:
    lukv_profile_budgets_ragged, lukv_score_ragged, lukv_select_gather_ragged against one single-sequence oracle run
    per sequence.  Budgets and offsets exact; selection and gather exact on the oracle's scores."""
    S, L, H, G, d, T, w, kp = 3, 2, 2, 4, 128, 2048, 32, 7
    lens, N, R = [2048, 1280, 700], 4, 9
    g = torch.Generator().manual_seed(12)
    q = torch.randn((S, L, H * G, w, d), generator=g).to(torch.bfloat16)
    k = torch.randn((S, L, H, T, d), generator=g).to(torch.bfloat16)
    v = torch.randn((S, L, H, T, d), generator=g).to(torch.bfloat16)
    rng = np.random.default_rng(12)
    ratios = np.linspace(0.1, 0.9, R).astype(np.float32)
    profile = np.sort(rng.random((R, N)).astype(np.float32), axis=0)        # per head non-decreasing in the ratio
    sigma = np.asarray([0.3, 0.55, 0.9], np.float32)                         # a grid point, between two, the last
    p = lukv.make_params(S, L, H, G, d, T, w, kp, torch.bfloat16, 2, n_sink=4, min_keep=0.02)
    budgets = torch.full((S, N), -1, dtype=torch.int32, device="cuda")
    offsets = torch.full((S * N + 1,), -1, dtype=torch.int32, device="cuda")
    lukv.lukv_profile_budgets_ragged(p, lens, torch.from_numpy(profile).cuda(), ratios, sigma, budgets, offsets)
    torch.cuda.synchronize()
    ref_b = np.concatenate([oracle.profile_budgets(profile, ratios, lens[s], w, sigma[s:s + 1], min_keep=0.02)[0]
                            for s in range(S)])
    ref_o = np.concatenate([[0], np.cumsum(ref_b.reshape(-1) + w)]).astype(np.int32)
    np.testing.assert_array_equal(budgets.cpu().numpy(), ref_b)
    np.testing.assert_array_equal(offsets.cpu().numpy(), ref_o)
    for s in range(S):
        assert ref_b[s].min() >= int(np.ceil(np.float32(0.02) * (lens[s] - w)))
    # scores of the ragged call, then eviction on the oracle's scores (so that near-ties cannot reorder positions)
    ws = lukv.alloc_workspace(p)
    scores = torch.zeros((S, N, T - w), dtype=torch.float32, device="cuda")
    lukv.lukv_score_ragged(p, lens, q.cuda(), k.cuda(), scores, ws)
    ref_scores = np.zeros((S, N, T - w), np.float32)
    for s, Ts in enumerate(lens):
        ref_scores[s, :, :Ts - w] = oracle.score(bits(q[s:s + 1]), bits(k[s:s + 1, :, :, :Ts].contiguous()), G, kp)[0]
    torch.cuda.synchronize()
    for s, Ts in enumerate(lens):
        assert_scores_close(scores.cpu().numpy()[s, :, :Ts - w], ref_scores[s, :, :Ts - w])
    rows = int(ref_o[-1])
    k_out = torch.zeros((rows, d), dtype=torch.bfloat16, device="cuda")
    v_out = torch.zeros((rows, d), dtype=torch.bfloat16, device="cuda")
    kept = torch.full((rows,), -1, dtype=torch.int32, device="cuda")
    lukv.lukv_select_gather_ragged(p, lens, torch.from_numpy(ref_scores).cuda(), budgets, offsets, k.cuda(), v.cuda(),
                                   k_out, v_out, kept, rows, ws)
    torch.cuda.synchronize()
    kept, ko, vo = kept.cpu().numpy(), bits(k_out), bits(v_out)
    for s, Ts in enumerate(lens):
        r0 = ref_o[s * N]
        rk, rv, rkept = oracle.select_gather(ref_scores[s, :, :Ts - w], ref_b[s], ref_o[s * N:(s + 1) * N + 1] - r0,
                                             bits(k[s, :, :, :Ts].contiguous()).reshape(N, Ts, d),
                                             bits(v[s, :, :, :Ts].contiguous()).reshape(N, Ts, d), w, n_sink=4)
        r1 = ref_o[(s + 1) * N]
        np.testing.assert_array_equal(kept[r0:r1], rkept)
        np.testing.assert_array_equal(ko[r0:r1], rk)
        np.testing.assert_array_equal(vo[r0:r1], rv)


def test_ragged_argument_errors():
    p = lukv.make_params(2, 1, 2, 2, 64, 256, 8, 3, "bf16", 17)
    f = torch.empty(1 << 20, dtype=torch.uint8, device="cuda")
    args = (f, f, f, f, [10, 10], f, f, f, f, f, 1 << 20, None, f)
    assert lukv.lukv_compress_ragged(p, [256, 8], *args, check=False) == lukv.ERR_INVALID_ARG       # not longer than the window
    assert lukv.lukv_compress_ragged(p, [256, 512], *args, check=False) == lukv.ERR_INVALID_ARG     # beyond the row stride
    assert lukv.lukv_compress_ragged(p, [256, 100], *args, check=False) == lukv.ERR_UNSUPPORTED     # 16 does not divide 100
    big = (f, f, f, f, [10, 2 * 2 * (64 - 8) + 1], f, f, f, f, f, 1 << 20, None, f)
    assert lukv.lukv_compress_ragged(p, [256, 64], *big, check=False) == lukv.ERR_BUDGET            # beyond N*n of that sequence
