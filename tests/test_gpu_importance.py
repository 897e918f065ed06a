"""GPU parity of the oracle importance (Sec. 4.1, Eq. "oracle_importance"; App. E) against the oracle, and the
offline chain importance -> curves -> profile on the GPU.  Attention weights are fp32 arithmetic on bf16 or
fp32 inputs, so the values carry the score tolerance (2e-3 relative, plus 1e-30 at the underflow edge)."""
import numpy as np
import pytest
import torch

from paper_2602_08585_b200 import lukv, synth
from gpu_helpers import SCORE_ATOL, SCORE_RTOL, bits

pytestmark = pytest.mark.gpu


def _inputs(S, L, H, G, d, T, Kmax, Dm, dtype, seed, scale=1.0):
    g = torch.Generator().manual_seed(seed)
    q = (torch.randn((S, L, H * G, Kmax, d), generator=g) * scale).to(dtype)
    k = (torch.randn((S, L, H, T, d), generator=g) * scale).to(dtype)
    v = torch.randn((S, L, H, T, d), generator=g).to(dtype)
    kd = (torch.randn((S, L, H, Kmax, d), generator=g) * scale).to(dtype)
    wo = (torch.randn((L, H * G, d, Dm), generator=g) / d ** 0.5).to(dtype)
    return q, k, v, kd, wo


def gpu_importance(p, Kmax, Dm, q, k, v, kd, wo, normalize):
    ws = torch.empty(lukv.lukv_importance_workspace_bytes(p, Kmax), dtype=torch.uint8, device="cuda")
    out = torch.full((p.batch, p.N, p.n), -7.0, dtype=torch.float32, device="cuda")
    lukv.lukv_oracle_importance(p, Kmax, Dm, q.cuda(), k.cuda(), v.cuda(), None if kd is None else kd.cuda(), wo.cuda(),
                                normalize, out, ws)
    torch.cuda.synchronize()
    return out.cpu().numpy()


def _close(got, ref):
    err = np.abs(got.astype(np.float64) - ref.astype(np.float64))
    bound = SCORE_RTOL * np.abs(ref.astype(np.float64)) + SCORE_ATOL
    assert np.all(err <= bound), f"worst relative error {(err / np.maximum(np.abs(ref), 1e-300)).max():.3e}"


SHAPES = [
    # S, L, H, G, d,   T,    w, Kmax, Dm, dtype,          decode keys, normalise
    (1, 1, 1, 1, 64, 2, 1, 1, 1, torch.float32, False, False),              # smallest legal problem
    (1, 2, 2, 1, 64, 77, 5, 3, 10, torch.float32, True, True),              # ragged everything
    (2, 1, 2, 4, 128, 1300, 32, 20, 200, torch.bfloat16, True, True),       # steps and projection width not multiples of the tiles
    (1, 1, 1, 7, 128, 600, 32, 33, 64, torch.bfloat16, True, False),        # GQA group 7: two chunks of query heads
    (1, 2, 3, 2, 64, 1025, 7, 16, 130, torch.bfloat16, False, True),        # no decode keys
    (1, 1, 2, 4, 128, 4000, 32, 8, 256, torch.bfloat16, True, True),        # the paper's calibration length
    # value norms on the tensor cores (bf16, d = 128): projection panels of 256 columns, chunks of 4096 positions
    (1, 2, 1, 2, 128, 700, 32, 4, 516, torch.bfloat16, False, True),        # three panels, the last one ragged
    (1, 1, 2, 1, 128, 300, 8, 3, 77, torch.bfloat16, True, False),          # odd width: the unvectorised panel writer
    (2, 1, 1, 2, 128, 4096 + 700, 32, 2, 264, torch.bfloat16, False, True), # two position chunks per head
]


@pytest.mark.parametrize("shape", SHAPES)
def test_importance_matches_oracle(oracle, shape):
    S, L, H, G, d, T, w, Kmax, Dm, dtype, with_kd, normalize = shape
    q, k, v, kd, wo = _inputs(S, L, H, G, d, T, Kmax, Dm, dtype, seed=T + Kmax, scale=1.5)
    p = lukv.make_params(S, L, H, G, d, T, w, 1, dtype, 2)
    got = gpu_importance(p, Kmax, Dm, q, k, v, kd if with_kd else None, wo, normalize)
    ref = oracle.importance(bits(q), bits(k), bits(v), bits(wo), G, w, k_dec=bits(kd) if with_kd else None,
                            normalize=normalize)
    _close(got, ref)
    if normalize:
        np.testing.assert_allclose(got.reshape(S, L, -1).sum(axis=2), 1.0, rtol=1e-4)


def test_value_norms_tensor_core_against_fp32_pipes(monkeypatch):
    """The two value-norm kernels (tensor cores; FP32 pipes, kept for other shapes) agree far inside the tolerance:
    bf16 products are exact in fp32 and both accumulate in fp32."""
    S, L, H, G, d, T, w, Kmax, Dm = 1, 2, 2, 4, 128, 2000, 32, 4, 1024
    q, k, v, kd, wo = _inputs(S, L, H, G, d, T, Kmax, Dm, torch.bfloat16, seed=21)
    p = lukv.make_params(S, L, H, G, d, T, w, 1, torch.bfloat16, 2)
    tc = gpu_importance(p, Kmax, Dm, q, k, v, kd, wo, False)
    monkeypatch.setenv("LUKV_FORCE_SIMT", "1")
    simt = gpu_importance(p, Kmax, Dm, q, k, v, kd, wo, False)
    np.testing.assert_allclose(tc, simt, rtol=2e-5, atol=1e-30)


def test_importance_at_the_benchmark_size_sampled_heads(oracle):
    """The size bench.py times (one calibration query of 4000 tokens, 256 KV heads x 4 query heads, 64 decode steps,
    model width 4096; the value norms run on the tensor cores over 1024 work items): two sampled heads against the
    oracle, without the per-layer normalisation (which would need every head of the layer)."""
    S, L, H, G, d, T, w, Kmax, Dm = 1, 32, 8, 4, 128, 4000, 32, 64, 4096
    g = torch.Generator(device="cuda").manual_seed(3)
    dt = torch.bfloat16
    q = torch.randn((S, L, H * G, Kmax, d), generator=g, device="cuda").to(dt)
    k = torch.randn((S, L, H, T, d), generator=g, device="cuda").to(dt)
    v = torch.randn((S, L, H, T, d), generator=g, device="cuda").to(dt)
    kd = torch.randn((S, L, H, Kmax, d), generator=g, device="cuda").to(dt)
    wo = (torch.randn((L, H * G, d, Dm), generator=g, device="cuda") / d ** 0.5).to(dt)
    p = lukv.make_params(S, L, H, G, d, T, w, 1, dt, 2)
    ws = torch.empty(lukv.lukv_importance_workspace_bytes(p, Kmax), dtype=torch.uint8, device="cuda")
    out = torch.full((S, L * H, T - w), -7.0, dtype=torch.float32, device="cuda")
    lukv.lukv_oracle_importance(p, Kmax, Dm, q, k, v, kd, wo, False, out, ws)
    torch.cuda.synchronize()
    for layer, h in [(0, 0), (19, 5)]:
        sub = lambda t, lo, hi: bits(t[:, layer:layer + 1, lo:hi].contiguous().cpu())
        ref = oracle.importance(sub(q, h * G, (h + 1) * G), sub(k, h, h + 1), sub(v, h, h + 1),
                                bits(wo[layer:layer + 1, h * G:(h + 1) * G].contiguous().cpu()), G, w,
                                k_dec=sub(kd, h, h + 1), normalize=False)
        _close(out[:, layer * H + h].cpu().numpy().reshape(ref.shape), ref)


def test_importance_argument_errors():
    p = lukv.make_params(1, 1, 2, 2, 64, 256, 8, 1, "bf16", 2)
    f = torch.empty(1024, dtype=torch.uint8, device="cuda")
    assert lukv.lukv_oracle_importance(p, 0, 8, f, f, f, None, f, True, f, f, check=False) == lukv.ERR_INVALID_ARG
    assert lukv.lukv_oracle_importance(p, 4, 0, f, f, f, None, f, True, f, f, check=False) == lukv.ERR_INVALID_ARG
    assert lukv.lukv_oracle_importance(p, 4, 8, None, f, f, None, f, True, f, f, check=False) == lukv.ERR_INVALID_ARG
    assert lukv.lukv_oracle_importance(p, 4, 8, f, f, f, None, f, True, f, f, check=False) == lukv.ERR_WORKSPACE_TOO_SMALL


def test_offline_chain_importance_to_profile(oracle):
    """The offline side of Sec. 4.1-4.3 on the GPU: oracle importance of every calibration query from its decode
    queries, the curves of the proxy ranking against it, the profile.  The curves use the oracle's proxy scores on
    both sides (near-ties in the scores must not reorder positions) and each side's own importance."""
    wl = synth.scaled(synth.CONFIGS["tiny"], S=3, T=512, P=513)       # 3 calibration queries, 4 heads, fp32, d = 64
    q_win, k, v = synth.gen_tensors(wl, "cpu")
    Kmax, Dm = 12, 96
    g = torch.Generator().manual_seed(11)
    q_dec = torch.randn((wl.S, wl.L, wl.H * wl.G, Kmax, wl.d), generator=g)
    k_dec = torch.randn((wl.S, wl.L, wl.H, Kmax, wl.d), generator=g)
    w_o = torch.randn((wl.L, wl.H * wl.G, wl.d, Dm), generator=g) / wl.d ** 0.5
    p = lukv.make_params(wl.S, wl.L, wl.H, wl.G, wl.d, wl.T, wl.w, wl.kp, wl.dtype, wl.P)
    imp_gpu = gpu_importance(p, Kmax, Dm, q_dec, k, v, k_dec, w_o, True)
    imp_ref = oracle.importance(bits(q_dec), bits(k), bits(v), bits(w_o), wl.G, wl.w, k_dec=bits(k_dec))
    _close(imp_gpu, imp_ref)
    s_ref = oracle.score(bits(q_win), bits(k), wl.G, wl.kp)
    c_ref = oracle.build_curves(s_ref.reshape(-1, wl.n), imp_ref.reshape(-1, wl.n), wl.T, wl.w, wl.P)
    curves = torch.empty((wl.S, wl.N, wl.P), dtype=torch.float32, device="cuda")
    lukv.lukv_build_curves(p, torch.from_numpy(s_ref).cuda(), torch.from_numpy(imp_gpu).cuda(), curves)
    total = c_ref[:, -1:].astype(np.float64)
    assert (np.abs(curves.cpu().numpy().reshape(-1, wl.P) - c_ref) / total).max() < SCORE_RTOL
    ratios = np.linspace(0.0, 1.0, 11).astype(np.float32)
    calib = lukv.make_params(1, wl.L, wl.H, 1, 64, wl.T, wl.w, 1, "fp32", wl.P)
    ws = torch.empty(lukv.lukv_profile_workspace_bytes(calib, wl.S, len(ratios)), dtype=torch.uint8, device="cuda")
    phi = torch.empty((len(ratios), wl.N), dtype=torch.float32, device="cuda")
    lukv.lukv_profile_build(calib, curves, wl.S, ratios, phi, ws)
    torch.cuda.synchronize()
    phi_ref = oracle.profile_build(c_ref.reshape(wl.S, wl.N, wl.P), wl.T, wl.w, ratios)
    # importance values that differ within the tolerance can move the cut of a query by a few tokens
    assert np.abs(phi.cpu().numpy() - phi_ref).max() < 0.02
    assert phi.cpu().numpy()[0].max() == 0.0 and phi.cpu().numpy()[-1].min() == 1.0
