"""The workspace-free allocation entry point against the regular one and against the oracle.

lukv_allocate_static serves callers that cannot allocate device memory when budgets are
needed (for instance a server whose memory belongs to its own pool): its scratch is a fixed
array inside the library.  It must produce exactly the budgets and offsets of lukv_allocate,
on consecutive calls that reuse the same scratch, and refuse problems beyond its limit.
This file sorts last so that a failure here cannot hide the other tests in a fail-fast run.
"""
import numpy as np
import pytest
import torch

from oracle import lukv_oracle
from paper_2602_08585_b200 import lukv, synth
from gpu_helpers import gpu_allocate


def _static_allocate(p, curves_np, budgets_in):
    curves = torch.from_numpy(np.ascontiguousarray(curves_np, dtype=np.float32)).cuda()
    budgets = torch.full((p.batch, p.N), -7, dtype=torch.int32, device="cuda")
    offsets = torch.full((p.batch * p.N + 1,), -7, dtype=torch.int32, device="cuda")
    lukv.lukv_allocate_static(p, curves, budgets_in, budgets, offsets)
    torch.cuda.synchronize()
    return budgets.cpu().numpy(), offsets.cpu().numpy()


@pytest.mark.gpu
def test_static_allocate_matches_allocate_on_two_calls_in_a_row():
    assert torch.cuda.is_available()
    # call 1: a large problem that fills much of the scratch; call 2: a smaller one with other
    # curves, which must not see anything the first call left behind
    big = synth.CONFIGS["llama8b_32k"]
    small = synth.scaled(synth.CONFIGS["batch8_16k_mixed"], S=3, L=4, H=2, T=2048, P=33)
    for wl in (big, small):
        p = lukv.make_params(wl.S, wl.L, wl.H, wl.G, wl.d, wl.T, wl.w, wl.kp, wl.dtype, wl.P)
        curves = synth.gen_curves(wl)
        b_static, o_static = _static_allocate(p, curves, wl.budgets())
        b_ref, o_ref = gpu_allocate(p, curves, wl.budgets())
        np.testing.assert_array_equal(b_static, b_ref)          # integer outputs: bit-exact
        np.testing.assert_array_equal(o_static, o_ref)
        np.testing.assert_array_equal(b_static.sum(axis=1), wl.budgets())
        b_orc, o_orc = lukv_oracle.allocate(curves, wl.T, wl.w, wl.budgets())
        np.testing.assert_array_equal(b_static, b_orc)
        np.testing.assert_array_equal(o_static, o_orc)


def test_static_allocate_rejects_sizes_beyond_its_scratch():
    # 300 heads x 1024 segments > 262144 gains: refused on the host, nothing is launched
    p = lukv.make_params(1, 300, 1, 1, 64, 4096, 32, 1, "bf16", 1025)

    class _Fake:
        def data_ptr(self):
            return 0x10000

    f = _Fake()
    assert lukv.lukv_allocate_static(p, f, [10], f, f, check=False) == lukv.ERR_WORKSPACE_TOO_SMALL
    ok = lukv.make_params(1, 2, 2, 1, 64, 256, 8, 1, "bf16", 17)
    assert lukv.lukv_allocate_static(ok, f, [-1], f, f, check=False) == lukv.ERR_BUDGET
    assert lukv.lukv_allocate_static(ok, None, [1], f, f, check=False) == lukv.ERR_INVALID_ARG
