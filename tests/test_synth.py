"""The seeded workload generator: determinism, shapes, and the stated recipe."""
import numpy as np
import torch

from paper_2602_08585_b200 import synth


def test_heads_are_reproducible_and_independent():
    wl = synth.CONFIGS["tiny"]
    a = synth.gen_head(wl, 0, 0, 1)
    b = synth.gen_head(wl, 0, 0, 1)
    c = synth.gen_head(wl, 0, 0, 2)
    for x, y in zip(a, b):
        assert torch.equal(x, y)
    assert not torch.equal(a[1], c[1])
    q, k, v = synth.gen_tensors(wl)
    assert q.shape == (1, 1, 4, 16, 64) and k.shape == (1, 1, 4, 1024, 64) and k.dtype == torch.float32
    assert torch.equal(k[0, 0, 1], a[1]) and torch.equal(q[0, 0, 1:2], a[0])


def test_distribution_and_outliers():
    wl = synth.scaled(synth.CONFIGS["llama8b_1layer_8k"], T=2048, P=33)
    qh, kh, vh = synth.gen_head(wl, 0, 0, 3)
    assert kh.dtype == torch.bfloat16 and kh.shape == (2048, 128)
    ch = synth.outlier_channels(wl, synth.head_index(wl, 0, 0, 3))
    assert len(set(ch)) == 4
    std = kh.float().std(dim=0)
    rest = [c for c in range(128) if c not in ch]
    assert abs(float(std[rest].mean()) - 1.0) < 0.05
    assert all(6.0 < float(std[c]) < 10.0 for c in ch)
    assert abs(float(vh.float().std()) - 1.0) < 0.02
    qstd = qh.float().reshape(-1, 128).std(dim=0)
    assert all(float(qstd[c]) > 4.0 for c in ch)


def test_needles_follow_the_window_query_mean():
    wl = synth.CONFIGS["tiny"]
    u = synth.head_index(wl, 0, 0, 0)
    qh, kh, _ = synth.gen_head(wl, 0, 0, 0)
    pos = synth.needle_positions(wl, u)
    assert len(pos) == len(set(pos)) == 8 and max(pos) < wl.n
    m = qh.double().reshape(-1, wl.d).mean(dim=0)
    dev = kh[pos].double() - 3.0 * m[None, :]
    assert 0.05 < float(dev.std()) < 0.2


def test_curves_and_budgets():
    wl = synth.CONFIGS["llama8b_32k"]
    c = synth.gen_curves(wl)
    assert c.shape == (256, 257) and c.dtype == np.float32 and np.all(c[:, 0] == 0)
    inc = np.diff(c.astype(np.float64), axis=1)
    assert np.all(inc > 0) and abs(inc.mean() - 1.4) < 0.05        # E = 0.8*1 + 0.2*3
    assert np.any(np.diff(inc, axis=1) > 0)                         # non-concave
    cc = synth.gen_curves(wl, concave=True)
    assert np.all(np.diff(np.diff(cc.astype(np.float64), axis=1), axis=1) <= 2e-4)      # up to fp32 rounding of the sums
    assert wl.budgets().tolist() == [1677721] and wl.total_rows() == 1685913
    w4 = synth.CONFIGS["batch8_16k_mixed"]
    assert w4.budgets().tolist() == [419430, 2097152] * 4 and w4.total_rows() == 10197400
    assert synth.CONFIGS["gqa7_128k"].total_rows() == 1471590
