"""ctypes front end of the CPU oracle (test infrastructure, not product code).

Loads ``liblukv_oracle.so`` (built from ``lukv_oracle.cpp`` by :func:`build`) and wraps
its entry points for numpy arrays.  Only the tests, the smoke check and the benchmark's
CPU-baseline leg may import this module; the CUDA library and its Python binding never do.

bf16 tensors are passed as ``uint16`` bit patterns (``dtype=0``), fp32 as ``float32``
(``dtype=1``).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lukv_oracle.cpp")
_LIB = os.path.join(_HERE, "liblukv_oracle.so")
_lib = None

BF16, FP32 = 0, 1


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (no fused multiply-add contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-O2", "-std=c++17", "-ffp-contract=off", "-shared", "-fPIC", _SRC, "-o", _LIB]
        subprocess.run(cmd, check=True)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.oracle_allocate.restype = ctypes.c_int
        _lib.oracle_compress.restype = ctypes.c_int
        _lib.oracle_profile_build.restype = ctypes.c_int
        _lib.oracle_profile_budgets.restype = ctypes.c_int
        for name in ("oracle_allocate_floor", "oracle_compress_ext", "oracle_profile_build_floor",
                     "oracle_profile_budgets_floor"):
            getattr(_lib, name).restype = ctypes.c_int
        _lib.oracle_exact_allocate.restype = ctypes.c_int
        _lib.oracle_floor_tokens.restype = ctypes.c_int64
        _lib.oracle_floor_tokens.argtypes = [ctypes.c_float, ctypes.c_int]
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _dtype_code(a: np.ndarray) -> int:
    if a.dtype == np.uint16:
        return BF16
    if a.dtype == np.float32:
        return FP32
    raise TypeError(f"oracle takes uint16 (bf16 bits) or float32, got {a.dtype}")


def _c(a, dtype=None):
    a = np.ascontiguousarray(a) if dtype is None else np.ascontiguousarray(a, dtype=dtype)
    return a


def window_softmax(q_head, k_head, scale: float = 0.0) -> np.ndarray:
    """Probabilities of one head: q_head [G][w][d], k_head [T][d] -> [G*w][T] float64."""
    q_head, k_head = _c(q_head), _c(k_head)
    G, w, d = q_head.shape
    T = k_head.shape[0]
    prob = np.empty((G * w, T), np.float64)
    lib().oracle_window_softmax(_p(q_head), _p(k_head), _dtype_code(k_head), G, w, d, T,
                                ctypes.c_float(scale), _p(prob))
    return prob


def score_head(q_head, k_head, kp: int, scale: float = 0.0):
    """One head -> (raw_full [T] float64, pooled [T-w] float32)."""
    q_head, k_head = _c(q_head), _c(k_head)
    G, w, d = q_head.shape
    T = k_head.shape[0]
    raw = np.empty(T, np.float64)
    pooled = np.empty(T - w, np.float32)
    lib().oracle_score_head(_p(q_head), _p(k_head), _dtype_code(k_head), G, w, d, T, kp,
                            ctypes.c_float(scale), _p(raw), _p(pooled))
    return raw, pooled


def score(q, k, G: int, kp: int, scale: float = 0.0) -> np.ndarray:
    """q [S][L][H*G][w][d], k [S][L][H][T][d] -> pooled scores [S][L*H][T-w] float32."""
    q, k = _c(q), _c(k)
    S, L, HG, w, d = q.shape
    H, T = k.shape[2], k.shape[3]
    assert HG == H * G
    out = np.empty((S, L * H, T - w), np.float32)
    lib().oracle_score(_p(q), _p(k), _dtype_code(k), S, L, H, G, d, T, w, kp, ctypes.c_float(scale), _p(out))
    return out


def max_pool(raw, kp: int) -> np.ndarray:
    raw = _c(raw, np.float64)
    out = np.empty_like(raw)
    lib().oracle_max_pool(_p(raw), raw.shape[0], kp, _p(out))
    return out


def hull(curves):
    """curves [N][P] float32 -> (gains float64 [N][P-1], gains rounded once to float32)."""
    curves = _c(curves, np.float32)
    N, P = curves.shape
    g64 = np.empty((N, P - 1), np.float64)
    g32 = np.empty((N, P - 1), np.float32)
    lib().oracle_hull(_p(curves), N, P, _p(g64), _p(g32))
    return g64, g32


def floor_tokens(min_keep: float, n: int) -> int:
    """Tokens every head keeps at least (App. E): ceil(min_keep * n)."""
    return int(lib().oracle_floor_tokens(ctypes.c_float(min_keep), int(n)))


def allocate(curves, T: int, w: int, budgets_in, min_keep: float = 0.0):
    """curves [N][P], budgets_in [S] -> (budgets int32 [S][N], offsets int32 [S*N+1]).
    min_keep > 0: every head first gets ceil(min_keep*(T-w)) tokens (App. E)."""
    curves = _c(curves, np.float32)
    budgets_in = _c(budgets_in, np.int64)
    N, P = curves.shape
    S = budgets_in.shape[0]
    budgets = np.empty((S, N), np.int32)
    offsets = np.empty(S * N + 1, np.int32)
    f = floor_tokens(min_keep, T - w)
    rc = lib().oracle_allocate_floor(_p(curves), N, P, T, w, S, _p(budgets_in), ctypes.c_int64(f), _p(budgets),
                                     _p(offsets))
    if rc != 0:
        raise ValueError("budget outside [N*floor, N*(T-w)]")
    return budgets, offsets


def select(pooled, b: int, n_sink: int = 0) -> np.ndarray:
    pooled = _c(pooled, np.float32)
    kept = np.empty(b, np.int32)
    lib().oracle_select_sink(_p(pooled), pooled.shape[0], b, int(n_sink), _p(kept))
    return kept


def select_gather(scores, budgets, offsets, k, v, w: int, n_sink: int = 0):
    """scores [U][n], budgets [U], offsets [U+1], k/v [U][T][d] -> (k_out, v_out, kept_idx)."""
    scores = _c(scores, np.float32)
    budgets = _c(budgets, np.int32).reshape(-1)
    offsets = _c(offsets, np.int32)
    k, v = _c(k), _c(v)
    U = budgets.shape[0]
    T, d = k.shape[-2], k.shape[-1]
    rows = int(offsets[-1])
    k_out = np.empty((rows, d), k.dtype)
    v_out = np.empty((rows, d), v.dtype)
    kept = np.empty(rows, np.int32)
    lib().oracle_select_gather_sink(_p(scores), _p(budgets), _p(offsets), _p(k), _p(v), _dtype_code(k), U, T, w, d,
                                    int(n_sink), _p(k_out), _p(v_out), _p(kept))
    return k_out, v_out, kept


def compress(q, k, v, curves, budgets_in, G: int, kp: int, scale: float = 0.0, n_sink: int = 0,
             min_keep: float = 0.0):
    """The whole path. Returns dict(k_out, v_out, kept_idx, budgets, offsets, scores)."""
    q, k, v = _c(q), _c(k), _c(v)
    curves = _c(curves, np.float32)
    budgets_in = _c(budgets_in, np.int64)
    S, L, HG, w, d = q.shape
    H, T = k.shape[2], k.shape[3]
    N, P = curves.shape
    assert HG == H * G and N == L * H
    rows = int(budgets_in.sum()) + S * N * w
    out = dict(
        k_out=np.empty((rows, d), k.dtype), v_out=np.empty((rows, d), v.dtype),
        kept_idx=np.empty(rows, np.int32), budgets=np.empty((S, N), np.int32),
        offsets=np.empty(S * N + 1, np.int32), scores=np.empty((S, N, T - w), np.float32))
    rc = lib().oracle_compress_ext(_p(q), _p(k), _p(v), _p(curves), _p(budgets_in), _dtype_code(k), S, L, H, G, d,
                               T, w, kp, P, ctypes.c_float(scale), int(n_sink), ctypes.c_float(min_keep),
                               _p(out["k_out"]), _p(out["v_out"]),
                               _p(out["kept_idx"]), _p(out["budgets"]), _p(out["offsets"]), _p(out["scores"]))
    if rc != 0:
        raise ValueError("budget outside [0, N*(T-w)]")
    return out


def compress_ragged(q, k, v, curves, budgets_in, ctx_lens, G: int, kp: int, scale: float = 0.0, n_sink: int = 0,
                    min_keep: float = 0.0):
    """A batch whose sequences have different context lengths (App. E applies the method to whatever context a
    request brings): k, v [S][L][H][T_max][d] with sequence s using the first ctx_lens[s] positions, its window
    being the last w of those.  By definition the result of one single-sequence call per sequence, concatenated:
    budgets [S][N], offsets [S*N+1] (running over all sequences), kept_idx / k_out / v_out in sequence order,
    scores as a list of [N][ctx_lens[s]-w] arrays."""
    q, k, v = _c(q), _c(k), _c(v)
    budgets_in = _c(budgets_in, np.int64)
    S = q.shape[0]
    parts = [compress(q[s:s + 1], np.ascontiguousarray(k[s:s + 1, :, :, :int(ctx_lens[s])]),
                      np.ascontiguousarray(v[s:s + 1, :, :, :int(ctx_lens[s])]), curves, budgets_in[s:s + 1], G, kp,
                      scale=scale, n_sink=n_sink, min_keep=min_keep) for s in range(S)]
    offsets, base = [np.zeros(1, np.int32)], 0
    for part in parts:
        offsets.append((part["offsets"][1:].astype(np.int64) + base).astype(np.int32))
        base += int(part["offsets"][-1])
    return dict(k_out=np.concatenate([part["k_out"] for part in parts]),
                v_out=np.concatenate([part["v_out"] for part in parts]),
                kept_idx=np.concatenate([part["kept_idx"] for part in parts]),
                budgets=np.concatenate([part["budgets"] for part in parts]),
                offsets=np.concatenate(offsets), scores=[part["scores"][0] for part in parts])


def profile_build(curves, T: int, w: int, ratios, min_keep: float = 0.0):
    """Offline profile (Sec. 4.3, Eq. "calibration_avg"). curves [Mq][N][P] -> profile [R][N] fp32."""
    curves = _c(curves, np.float32)
    ratios = _c(ratios, np.float32)
    Mq, N, P = curves.shape
    R = ratios.shape[0]
    profile = np.empty((R, N), np.float32)
    rc = lib().oracle_profile_build_floor(_p(curves), Mq, N, P, T, w, _p(ratios), R, ctypes.c_float(min_keep),
                                          _p(profile))
    if rc != 0:
        raise ValueError("ratio outside [0, 1]")
    return profile


def profile_budgets(profile, ratios, T: int, w: int, sigma, min_keep: float = 0.0):
    """Online lookup + budgeting (Sec. 4.3). Returns (budgets [S][N] int32, offsets [S*N+1] int32)."""
    profile = _c(profile, np.float32)
    ratios = _c(ratios, np.float32)
    sigma = _c(sigma, np.float32).reshape(-1)
    R, N = profile.shape
    S = sigma.shape[0]
    budgets = np.empty((S, N), np.int32)
    offsets = np.empty(S * N + 1, np.int32)
    rc = lib().oracle_profile_budgets_floor(_p(profile), _p(ratios), R, N, T, w, _p(sigma), S,
                                            ctypes.c_float(min_keep), _p(budgets), _p(offsets))
    if rc != 0:
        raise ValueError("sigma outside the ratio grid, or grid not strictly ascending")
    return budgets, offsets


def build_curves(scores, importance, T: int, w: int, P: int, n_sink: int = 0) -> np.ndarray:
    """Utility curves of the proxy ranking: scores, importance [heads][n] -> curves [heads][P] fp32."""
    scores = _c(scores, np.float32)
    importance = _c(importance, np.float32)
    heads, n = scores.shape
    assert n == T - w and importance.shape == scores.shape and T % (P - 1) == 0
    curves = np.empty((heads, P), np.float32)
    lib().oracle_build_curves(_p(scores), _p(importance), heads, T, w, P, int(n_sink), _p(curves))
    return curves


def importance(q_dec, k, v, w_o, G: int, w: int, k_dec=None, scale: float = 0.0, normalize: bool = True) -> np.ndarray:
    """Oracle importance (Sec. 4.1): q_dec [S][L][H*G][Kmax][d], k, v [S][L][H][T][d], w_o [L][H*G][d][Dm],
    k_dec [S][L][H][Kmax][d] or None -> importance [S][L*H][T-w] float32."""
    q_dec, k, v, w_o = _c(q_dec), _c(k), _c(v), _c(w_o)
    k_dec = None if k_dec is None else _c(k_dec)
    S, L, HG, Kmax, d = q_dec.shape
    H, T = k.shape[2], k.shape[3]
    Dm = w_o.shape[3]
    assert HG == H * G and v.shape == k.shape and w_o.shape == (L, H * G, d, Dm)
    assert k_dec is None or k_dec.shape == (S, L, H, Kmax, d)
    out = np.empty((S, L * H, T - w), np.float32)
    lib().oracle_importance(_p(q_dec), _p(k), _p(v), _p(k_dec), _p(w_o), _dtype_code(k), S, L, H, G, d, T, w, Kmax, Dm,
                            ctypes.c_float(scale), int(bool(normalize)), _p(out))
    return out


def keydiff(k, w: int) -> np.ndarray:
    """KeyDiff proxy scores: k [S][L][H][T][d] -> [S][L*H][T-w] float32 (negated cosine similarity of every
    rankable key with the mean of the head's unit-normalised keys)."""
    k = _c(k)
    S, L, H, T, d = k.shape
    out = np.empty((S, L * H, T - w), np.float32)
    lib().oracle_keydiff(_p(k), _dtype_code(k), S * L * H, T, w, d, _p(out))
    return out


def exact_allocate(curves, T: int, w: int, budgets_in):
    """Exact allocation on token-resolution curves [N][T+1] -> (budgets [S][N] int32, optimum values [S] float64)."""
    curves = _c(curves, np.float32)
    budgets_in = _c(budgets_in, np.int64)
    N, P = curves.shape
    S = budgets_in.shape[0]
    budgets = np.empty((S, N), np.int32)
    values = np.empty(S, np.float64)
    rc = lib().oracle_exact_allocate(_p(curves), N, P, T, w, S, _p(budgets_in), _p(budgets), _p(values))
    if rc != 0:
        raise ValueError("needs token-resolution curves (P = T+1) and budgets in [0, N*(T-w)]")
    return budgets, values
