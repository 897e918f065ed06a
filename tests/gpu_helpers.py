"""Shared helpers of the GPU parity tests: calls go through the C ABI binding only."""
import numpy as np
import torch

from paper_2602_08585_b200 import lukv, synth

SCORE_RTOL = 2e-3      # max relative error of the scores (bf16 in, fp32 accumulate)
SCORE_ATOL = 1e-30     # scores this small sit at the fp32 underflow edge


def params_of(wl: synth.Workload) -> lukv.Params:
    return lukv.make_params(wl.S, wl.L, wl.H, wl.G, wl.d, wl.T, wl.w, wl.kp, wl.dtype, wl.P)


def gpu_score(p, q, k):
    ws = lukv.alloc_workspace(p)
    scores = torch.empty((p.batch, p.N, p.n), dtype=torch.float32, device="cuda")
    lukv.lukv_score(p, q, k, scores, ws)
    torch.cuda.synchronize()
    return scores


def gpu_allocate(p, curves_np, budgets_in):
    ws = lukv.alloc_workspace(p)
    curves = torch.from_numpy(np.ascontiguousarray(curves_np, dtype=np.float32)).cuda()
    budgets = torch.full((p.batch, p.N), -7, dtype=torch.int32, device="cuda")
    offsets = torch.full((p.batch * p.N + 1,), -7, dtype=torch.int32, device="cuda")
    lukv.lukv_allocate(p, curves, budgets_in, budgets, offsets, ws)
    torch.cuda.synchronize()
    return budgets.cpu().numpy(), offsets.cpu().numpy()


def gpu_select_gather(p, scores, budgets, offsets, k, v, rows, pad_rows=0):
    """Returns (k_out, v_out, kept_idx) with `pad_rows` canary rows after the real ones."""
    ws = lukv.alloc_workspace(p)
    dt = k.dtype
    k_out = torch.zeros((rows + pad_rows, p.head_dim), dtype=dt, device="cuda")
    v_out = torch.zeros((rows + pad_rows, p.head_dim), dtype=dt, device="cuda")
    kept = torch.full((rows + pad_rows,), -1, dtype=torch.int32, device="cuda")
    lukv.lukv_select_gather(p, scores, budgets, offsets, k, v, k_out, v_out, kept, rows, ws)
    torch.cuda.synchronize()
    return k_out, v_out, kept


def gpu_compress(p, q, k, v, curves_np, budgets_in):
    ws = lukv.alloc_workspace(p)
    out = lukv.Outputs(p, budgets_in)
    curves = torch.from_numpy(np.ascontiguousarray(curves_np, dtype=np.float32)).cuda()
    lukv.lukv_compress(p, q, k, v, curves, budgets_in, out.k_out, out.v_out, out.kept_idx, out.budgets, out.offsets,
                       out.rows, out.dev_status, ws)
    torch.cuda.synchronize()
    assert int(out.dev_status.item()) == 0
    return out


def assert_scores_close(gpu: np.ndarray, ref: np.ndarray):
    err = np.abs(gpu.astype(np.float64) - ref.astype(np.float64))
    bound = SCORE_RTOL * np.abs(ref.astype(np.float64)) + SCORE_ATOL
    bad = err > bound
    assert not bad.any(), (f"{bad.sum()} of {bad.size} scores outside tolerance; worst rel err "
                           f"{(err / np.maximum(np.abs(ref), 1e-300)).max():.3e}")


def kept_agreement(kept_gpu, kept_ref, offsets, budgets, scores_ref, n_sink=0):
    """Fraction of the oracle's kept (non-window) positions that the GPU path kept too; every
    position in the symmetric difference must sit within the score tolerance of the oracle's
    threshold score of that head (with attention sinks: of its scored, non-sink positions)."""
    budgets = budgets.reshape(-1)
    scores_ref = scores_ref.reshape(budgets.shape[0], -1)
    same = total = 0
    for u, b in enumerate(budgets):
        if b == 0:
            continue
        o = offsets[u]
        g = kept_gpu[o:o + b]
        r = kept_ref[o:o + b]
        assert np.all(np.diff(g) > 0) and g.min() >= 0 and g.max() < scores_ref.shape[1]
        inter = np.intersect1d(g, r, assume_unique=True)
        same += len(inter)
        total += b
        diff = np.setxor1d(g, r, assume_unique=True)
        if len(diff):
            assert b > n_sink and diff.min() >= n_sink, f"head {u}: a sink position differs"
            t = np.sort(scores_ref[u][n_sink:])[::-1][b - n_sink - 1].astype(np.float64)
            gap = np.abs(scores_ref[u][diff].astype(np.float64) - t)
            assert np.all(gap <= 2 * (SCORE_RTOL * t + SCORE_ATOL)), f"head {u}: mismatch away from the threshold"
    return same / max(total, 1)


def bits(t: torch.Tensor) -> np.ndarray:
    return synth.to_numpy_bits(t)
