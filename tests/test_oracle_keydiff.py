"""Pins of the oracle's KeyDiff proxy (pi_2 of Sec. 5.1; recent window 1 in App. E).  The paper only names the
metric; the formula is the one of the method's own publication: score_j = -cos(k_j, mean of the head's unit keys).
Pinned by library routines (torch normalisation and cosine similarity), closed forms and invariances."""
import numpy as np
import torch
import torch.nn.functional as F


def test_against_library_cosine_similarity(oracle):
    rng = np.random.default_rng(0)
    S, L, H, T, d, w = 2, 2, 3, 97, 16, 1
    k = rng.standard_normal((S, L, H, T, d)).astype(np.float32) * rng.uniform(0.1, 10.0, size=(S, L, H, T, 1)).astype(np.float32)
    got = oracle.keydiff(k, w)
    kt = torch.from_numpy(k).double()
    anchor = F.normalize(kt, dim=-1).mean(dim=3, keepdim=True)
    want = -F.cosine_similarity(kt, anchor, dim=-1)[..., : T - w].reshape(S, L * H, T - w)
    np.testing.assert_allclose(got, want.numpy(), rtol=1e-6, atol=1e-7)


def test_closed_forms(oracle):
    d, T = 8, 11
    e0, e1 = np.eye(d, dtype=np.float32)[0], np.eye(d, dtype=np.float32)[1]
    same = np.tile(3.0 * e0, (1, 1, 1, T, 1)).astype(np.float32)
    np.testing.assert_allclose(oracle.keydiff(same, 1), -1.0, atol=1e-7)          # every key is the mean direction
    odd = same.copy()
    odd[0, 0, 0, 4] = 5.0 * e1                                                     # one key orthogonal to the rest
    got = oracle.keydiff(odd, 1)[0, 0]
    a = np.array([(T - 1) / T, 1 / T])                                             # anchor in the (e0, e1) plane
    cos_rest, cos_odd = a[0] / np.linalg.norm(a), a[1] / np.linalg.norm(a)
    want = np.full(T - 1, -cos_rest)
    want[4] = -cos_odd
    np.testing.assert_allclose(got, want, rtol=1e-6)
    assert got.argmax() == 4                                                       # the odd key is the first to be kept
    # two opposite groups of different size: the minority scores +1, the majority -1
    two = same.copy()
    two[0, 0, 0, :3] = -2.0 * e0
    got = oracle.keydiff(two, 1)[0, 0]
    np.testing.assert_allclose(got[:3], 1.0, atol=1e-7)
    np.testing.assert_allclose(got[3:], -1.0, atol=1e-7)


def test_invariances_and_window(oracle):
    rng = np.random.default_rng(1)
    k = rng.standard_normal((1, 1, 2, 40, 8)).astype(np.float32)
    base = oracle.keydiff(k, 1)
    scaled = k.copy()
    scaled[0, 0, :, 7] *= 16.0                    # rescaling one key changes nothing: only directions enter
    scaled[0, 0, :, 20] *= 0.25
    np.testing.assert_allclose(oracle.keydiff(scaled, 1), base, rtol=1e-6, atol=1e-7)
    np.testing.assert_allclose(oracle.keydiff(-k, 1), base, rtol=1e-6, atol=1e-7)      # a common sign flip cancels
    # a wider recent window only drops trailing positions (the mean still runs over all T keys)
    np.testing.assert_array_equal(oracle.keydiff(k, 5), base[..., : 40 - 5])
    zero = k.copy()
    zero[0, 0, 0, 3] = 0.0                        # a zero key has no direction: its score is 0, nothing is NaN
    got = oracle.keydiff(zero, 1)
    assert np.isfinite(got).all() and got[0, 0, 3] == 0.0
