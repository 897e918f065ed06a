"""GPU parity of the offline profile and the online lookup/budgeting (Sec. 4.3) against the oracle.

The profile is a floating-point mean taken in the same order and precision on both sides and
is compared bit for bit; the budgets are integers and must be equal."""
import numpy as np
import pytest
import torch

from paper_2602_08585_b200 import lukv, synth

pytestmark = pytest.mark.gpu


def _calib_params(L, H, T, w, P):
    return lukv.make_params(1, L, H, 1, 64, T, w, 1, "fp32", P)


def gpu_profile_build(calib, curves_np, ratios):
    Mq = curves_np.shape[0]
    R = len(ratios)
    ws = torch.empty(lukv.lukv_profile_workspace_bytes(calib, Mq, R), dtype=torch.uint8, device="cuda")
    curves = torch.from_numpy(np.ascontiguousarray(curves_np, dtype=np.float32)).cuda()
    profile = torch.full((R, calib.N), -7.0, dtype=torch.float32, device="cuda")
    lukv.lukv_profile_build(calib, curves, Mq, ratios, profile, ws)
    torch.cuda.synchronize()
    return profile.cpu().numpy()


def gpu_profile_budgets(p, profile_np, ratios, sigma):
    profile = torch.from_numpy(np.ascontiguousarray(profile_np, dtype=np.float32)).cuda()
    budgets = torch.full((p.batch, p.N), -7, dtype=torch.int32, device="cuda")
    offsets = torch.full((p.batch * p.N + 1,), -7, dtype=torch.int32, device="cuda")
    lukv.lukv_profile_budgets(p, profile, ratios, sigma, budgets, offsets)
    torch.cuda.synchronize()
    return budgets.cpu().numpy(), offsets.cpu().numpy()


def _rough(rng, Mq, N, P):
    inc = rng.exponential(size=(Mq, N, P - 1)) * np.where(rng.random((Mq, N, P - 1)) < 0.2, 3.0, 1.0)
    U = np.zeros((Mq, N, P), np.float32)
    U[:, :, 1:] = np.cumsum(inc, axis=2)
    return U


def test_profile_small_token_resolution(oracle):
    L, H, T, w = 2, 4, 256, 16
    U = synth.gen_calibration_curves(101, 3, L * H, T)
    ratios = np.linspace(0.0, 1.0, 21).astype(np.float32)
    got = gpu_profile_build(_calib_params(L, H, T, w, T + 1), U, ratios)
    np.testing.assert_array_equal(got, oracle.profile_build(U, T, w, ratios))
    np.testing.assert_array_equal(got[0], 0.0)
    np.testing.assert_array_equal(got[-1], 1.0)


def test_profile_coarse_curves_many_ratios_many_heads(oracle):
    rng = np.random.default_rng(4)
    L, H, T, w, P = 3, 100, 1024, 16, 33     # 32 tokens per segment, ragged last segment, 300 heads
    U = _rough(rng, 5, L * H, P)
    U[2] = U[2, 0]                           # one query whose heads are all alike (every gain ties)
    ratios = np.sort(rng.random(40)).astype(np.float32)   # more grid points than one launch takes
    ratios[0], ratios[-1] = 0.0, 1.0
    got = gpu_profile_build(_calib_params(L, H, T, w, P), U, ratios)
    np.testing.assert_array_equal(got, oracle.profile_build(U, T, w, ratios))


def test_profile_single_query_single_ratio(oracle):
    rng = np.random.default_rng(6)
    U = _rough(rng, 1, 5, 9)
    for rho in (0.0, 0.37, 1.0):
        ratios = np.array([rho], np.float32)
        got = gpu_profile_build(_calib_params(1, 5, 64, 5, 9), U, ratios)
        np.testing.assert_array_equal(got, oracle.profile_build(U, 64, 5, ratios))


def test_profile_paper_size(oracle):
    # the paper's default calibration set: a context of about 4,000 tokens, 30 queries; a model of
    # 32 layers x 8 KV heads; ratios 0.01 .. 0.99
    L, H, T, w, Mq = 32, 8, 4000, 32, 30
    U = synth.gen_calibration_curves(synth.BASE_SEED, Mq, L * H, T)
    ratios = (np.arange(1, 100) / 100.0).astype(np.float32)
    got = gpu_profile_build(_calib_params(L, H, T, w, T + 1), U, ratios)
    ref = oracle.profile_build(U, T, w, ratios)
    np.testing.assert_array_equal(got, ref)
    assert (np.diff(got.astype(np.float64), axis=0) >= -1e-7).all()


def test_budgets_from_profile_bit_exact(oracle):
    rng = np.random.default_rng(8)
    N, Tc, wc = 256, 512, 32
    U = synth.gen_calibration_curves(55, 4, N, Tc)
    ratios = (np.arange(0, 51) / 50.0).astype(np.float32)
    phi = oracle.profile_build(U, Tc, wc, ratios)
    S, T, w = 40, 32768, 32                  # more sequences than one launch takes
    sigma = rng.random(S).astype(np.float32)
    sigma[:6] = [0.0, 1.0, ratios[7], ratios[8], np.nextafter(ratios[8], np.float32(0)), 0.5]
    p = lukv.make_params(S, 32, 8, 4, 128, T, w, 7, "bf16", 257)
    b, off = gpu_profile_budgets(p, phi, ratios, sigma)
    b_ref, off_ref = oracle.profile_budgets(phi, ratios, T, w, sigma)
    np.testing.assert_array_equal(b, b_ref)
    np.testing.assert_array_equal(off, off_ref)
    # a one-point grid, and a context shorter than the calibration one
    b, off = gpu_profile_budgets(lukv.make_params(1, 32, 8, 4, 128, 300, 32, 7, "bf16", 3), phi[20:21], ratios[20:21],
                                 ratios[20:21])
    b_ref, off_ref = oracle.profile_budgets(phi[20:21], ratios[20:21], 300, 32, ratios[20:21])
    np.testing.assert_array_equal(b, b_ref)
    np.testing.assert_array_equal(off, off_ref)


def test_online_mode_end_to_end(oracle):
    # Sec. 4.3 online execution on the GPU: lookup + budgeting, then eviction (selection + gather) by
    # the proxy scores; the scores fed to both sides are the oracle's, so the kept sets must be equal
    wl = synth.CONFIGS["tiny"]
    q, k, v = synth.gen_tensors(wl)
    U = synth.gen_calibration_curves(9, 3, wl.N, 128)
    ratios = np.linspace(0.0, 1.0, 11).astype(np.float32)
    calib = _calib_params(wl.L, wl.H, 128, wl.w, 129)
    phi = gpu_profile_build(calib, U, ratios)
    np.testing.assert_array_equal(phi, oracle.profile_build(U, 128, wl.w, ratios))
    sigma = np.array([0.83], np.float32)
    p = lukv.make_params(wl.S, wl.L, wl.H, wl.G, wl.d, wl.T, wl.w, wl.kp, wl.dtype, wl.P)
    b, off = gpu_profile_budgets(p, phi, ratios, sigma)
    b_ref, off_ref = oracle.profile_budgets(phi, ratios, wl.T, wl.w, sigma)
    np.testing.assert_array_equal(b, b_ref)
    np.testing.assert_array_equal(off, off_ref)
    qn, kn, vn = (synth.to_numpy_bits(t) for t in (q, k, v))
    scores = oracle.score(qn, kn, wl.G, wl.kp)
    rows = int(off[-1])
    ws = lukv.alloc_workspace(p)
    k_out = torch.zeros((rows, wl.d), dtype=k.dtype, device="cuda")
    v_out = torch.zeros((rows, wl.d), dtype=k.dtype, device="cuda")
    kept = torch.full((rows,), -1, dtype=torch.int32, device="cuda")
    lukv.lukv_select_gather(p, torch.from_numpy(scores).cuda(), torch.from_numpy(b).cuda(),
                            torch.from_numpy(off).cuda(), k.cuda(), v.cuda(), k_out, v_out, kept, rows, ws)
    torch.cuda.synchronize()
    k_ref, v_ref, kept_ref = oracle.select_gather(scores, b_ref, off_ref, kn, vn, wl.w)
    np.testing.assert_array_equal(kept.cpu().numpy(), kept_ref)
    np.testing.assert_array_equal(synth.to_numpy_bits(k_out), k_ref)
    np.testing.assert_array_equal(synth.to_numpy_bits(v_out), v_ref)
    # the scores the library computes itself rank the same positions (up to near-ties)
    s_gpu = torch.empty((p.batch, p.N, p.n), dtype=torch.float32, device="cuda")
    lukv.lukv_score(p, q.cuda(), k.cuda(), s_gpu, ws)
    kept2 = torch.full((rows,), -1, dtype=torch.int32, device="cuda")
    lukv.lukv_select_gather(p, s_gpu, torch.from_numpy(b).cuda(), torch.from_numpy(off).cuda(), k.cuda(), v.cuda(),
                            k_out, v_out, kept2, rows, ws)
    torch.cuda.synchronize()
    agree = (kept2.cpu().numpy() == kept_ref).mean()
    assert agree >= 0.99, agree
