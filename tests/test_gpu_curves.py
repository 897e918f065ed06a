"""GPU parity of the curve builder (Sec. 3.2, Eq. "head_loss_def") against the oracle, and the whole offline
chain scores -> curves -> profile.  Curve points are fp64 sums rounded to fp32; the two sides associate the
sums differently, so a point may differ by one rounding of the last bit: relative 2e-7."""
import numpy as np
import pytest
import torch

from paper_2602_08585_b200 import lukv, synth

pytestmark = pytest.mark.gpu
RTOL = 2e-7


def gpu_curves(p, scores, imp):
    curves = torch.full((p.batch, p.N, p.curve_points), -7.0, dtype=torch.float32, device="cuda")
    lukv.lukv_build_curves(p, torch.from_numpy(scores).cuda(), torch.from_numpy(imp).cuda(), curves)
    torch.cuda.synchronize()
    return curves.cpu().numpy()


def _case(oracle, S, L, H, T, w, P, n_sink=0, seed=0, ties=False):
    rng = np.random.default_rng(seed)
    N, n = L * H, T - w
    scores = rng.random((S, N, n)).astype(np.float32)
    if ties:
        scores = np.round(scores * 8).astype(np.float32) / 8          # nine distinct values: long runs of equals
    imp = rng.exponential(size=(S, N, n)).astype(np.float32)
    p = lukv.make_params(S, L, H, 1, 64, T, w, 1, "fp32", P, n_sink=n_sink)
    got = gpu_curves(p, scores, imp)
    ref = oracle.build_curves(scores.reshape(S * N, n), imp.reshape(S * N, n), T, w, P, n_sink=n_sink)
    np.testing.assert_allclose(got.reshape(S * N, P), ref, rtol=RTOL, atol=0)
    assert (got[..., 0] == 0).all()
    return got


def test_small_and_ragged(oracle):
    _case(oracle, 1, 1, 3, 48, 6, 9)                       # n = 42 (not a multiple of 4), clipped last segment
    _case(oracle, 2, 2, 2, 64, 5, 65, n_sink=4, seed=1)    # token resolution, n = 59, sinks
    _case(oracle, 1, 1, 2, 64, 63, 3, seed=2)              # one rankable position


def test_ties_follow_the_position_rule(oracle):
    _case(oracle, 1, 2, 3, 512, 16, 33, seed=3, ties=True)
    _case(oracle, 1, 1, 2, 512, 16, 513, n_sink=4, seed=4, ties=True)


def test_calibration_size(oracle):
    # the paper's calibration context: about 4,000 tokens at token resolution; 64 heads, 2 queries
    got = _case(oracle, 2, 8, 8, 4000, 32, 4001, n_sink=4, seed=5)
    assert (np.diff(got.astype(np.float64), axis=-1) >= 0).all()


def test_beyond_the_sorting_kernel(oracle):
    # more than 16384 positions: ranks by counting instead of the shared-memory sort
    _case(oracle, 1, 1, 2, 20000, 32, 126, n_sink=4, seed=6, ties=True)


def test_too_long_contexts_are_refused():
    p = lukv.make_params(1, 1, 1, 1, 64, 32768, 32, 1, "fp32", 257)
    f = torch.empty(1, device="cuda")
    assert lukv.lukv_build_curves(p, f, f, f, check=False) == lukv.ERR_UNSUPPORTED


def test_offline_chain_scores_to_profile(oracle):
    """Proxy scores of each calibration query (its own observation window), the curves of that ranking
    against a given importance, then the profile: every step on the GPU, against the same chain in the oracle.
    The curves are built from the oracle's scores on both sides, so that near-ties in the scores cannot
    reorder positions; the GPU's own scores are checked to give nearly the same curves."""
    wl = synth.scaled(synth.CONFIGS["tiny"], S=3, T=512, P=513)       # 3 calibration queries, 4 heads
    q, k, v = synth.gen_tensors(wl, "cuda")
    p = lukv.make_params(wl.S, wl.L, wl.H, wl.G, wl.d, wl.T, wl.w, wl.kp, wl.dtype, wl.P, n_sink=4)
    rng = np.random.default_rng(6)
    imp = rng.exponential(size=(wl.S, wl.N, wl.n)).astype(np.float32)
    s_ref = oracle.score(synth.to_numpy_bits(q), synth.to_numpy_bits(k), wl.G, wl.kp)
    c_ref = oracle.build_curves(s_ref.reshape(-1, wl.n), imp.reshape(-1, wl.n), wl.T, wl.w, wl.P, n_sink=4)
    c_gpu = gpu_curves(p, s_ref, imp)
    np.testing.assert_allclose(c_gpu.reshape(-1, wl.P), c_ref, rtol=RTOL)
    # profile from the curves (the GPU's own curves on the GPU, the oracle's in the oracle)
    ratios = np.linspace(0.0, 1.0, 21).astype(np.float32)
    calib = lukv.make_params(1, wl.L, wl.H, 1, 64, wl.T, wl.w, 1, "fp32", wl.P)
    ws = torch.empty(lukv.lukv_profile_workspace_bytes(calib, wl.S, len(ratios)), dtype=torch.uint8, device="cuda")
    phi = torch.empty((len(ratios), wl.N), dtype=torch.float32, device="cuda")
    lukv.lukv_profile_build(calib, torch.from_numpy(c_gpu).cuda(), wl.S, ratios, phi, ws)
    torch.cuda.synchronize()
    phi_ref = oracle.profile_build(c_ref.reshape(wl.S, wl.N, wl.P), wl.T, wl.w, ratios)
    # a curve point that differs in its last bit can move a token between two heads of one query
    assert np.abs(phi.cpu().numpy() - phi_ref).max() <= 2.0 / wl.n / wl.S + 1e-7
    # the library's own scores: same curves up to the positions whose scores nearly tie
    ws_s = lukv.alloc_workspace(p)
    s_gpu = torch.empty((wl.S, wl.N, wl.n), dtype=torch.float32, device="cuda")
    lukv.lukv_score(p, q, k, s_gpu, ws_s)
    c_own = gpu_curves(p, s_gpu.cpu().numpy(), imp)
    total = c_ref[:, -1:].astype(np.float64)
    assert (np.abs(c_own.reshape(-1, wl.P) - c_ref) / total).max() < 2e-3
