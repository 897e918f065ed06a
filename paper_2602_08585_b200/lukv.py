"""Thin ctypes binding of liblukv.so: same names as the C ABI (include/lukv.h), argument
marshalling only.  Every step of the path runs in the library's CUDA kernels; torch is
used for device memory and the current stream.  There is no CPU fallback: if the shared
library is missing the import of the entry points raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np
import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "liblukv.so")

OK = 0
ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_BUDGET, ERR_WORKSPACE_TOO_SMALL = -1, -2, -3, -4
ERR_OUTPUT_TOO_SMALL, ERR_CUDA, ERR_TIMEOUT = -5, -6, -7
DTYPE_BF16, DTYPE_FP32 = 0, 1
FLAG_KEYDIFF = 1  # params.flags: stage (a) is the KeyDiff metric

EXPORTS = ("lukv_workspace_bytes", "lukv_score", "lukv_allocate", "lukv_select_gather", "lukv_compress",
           "lukv_strerror", "lukv_last_launch_count", "lukv_compress_profile", "lukv_allocate_static",
           "lukv_profile_workspace_bytes", "lukv_profile_build", "lukv_profile_budgets", "lukv_build_curves", "lukv_exact_workspace_bytes",
           "lukv_exact_allocate", "lukv_importance_workspace_bytes", "lukv_oracle_importance", "lukv_score_ragged",
           "lukv_compress_ragged", "lukv_score_keydiff", "lukv_select_gather_ragged",
           "lukv_profile_budgets_ragged")


class Params(ctypes.Structure):
    """Mirror of lukv_params_t."""
    _fields_ = [("batch", ctypes.c_int32), ("n_layers", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
                ("gqa_group", ctypes.c_int32), ("head_dim", ctypes.c_int32), ("ctx_len", ctypes.c_int32),
                ("window", ctypes.c_int32), ("pool_kernel", ctypes.c_int32), ("dtype", ctypes.c_int32),
                ("curve_points", ctypes.c_int32), ("softmax_scale", ctypes.c_float), ("flags", ctypes.c_int32),
                ("n_sink", ctypes.c_int32), ("min_keep", ctypes.c_float)]

    @property
    def N(self):
        return self.n_layers * self.n_kv_heads

    @property
    def n(self):
        return self.ctx_len - self.window


class KernelTime(ctypes.Structure):
    """Mirror of lukv_kernel_time_t."""
    _fields_ = [("name", ctypes.c_char_p), ("ms", ctypes.c_float)]


class LukvError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {strerror(code)} ({code})")


_lib: Optional[ctypes.CDLL] = None


def lib() -> ctypes.CDLL:
    """Loads liblukv.so; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2602_08585_b200.build` "
                               "(the LU-KV path has no CPU or PyTorch fallback)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i64, sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_size_t
        pp = ctypes.POINTER(Params)
        L.lukv_workspace_bytes.argtypes = [pp, ctypes.POINTER(sz)]
        L.lukv_score.argtypes = [pp, vp, vp, vp, vp, sz, vp]
        L.lukv_allocate.argtypes = [pp, vp, vp, vp, vp, vp, sz, vp]
        L.lukv_select_gather.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, vp, i64, vp, sz, vp]
        L.lukv_compress.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, i64, vp, vp, sz, vp]
        L.lukv_compress_profile.argtypes = L.lukv_compress.argtypes + [ctypes.POINTER(KernelTime), ctypes.c_int,
                                                                       ctypes.POINTER(ctypes.c_int)]
        L.lukv_allocate_static.argtypes = [pp, vp, vp, vp, vp, vp]
        L.lukv_profile_workspace_bytes.argtypes = [pp, ctypes.c_int32, ctypes.c_int32, ctypes.POINTER(sz)]
        L.lukv_profile_build.argtypes = [pp, vp, ctypes.c_int32, vp, ctypes.c_int32, vp, vp, sz, vp]
        L.lukv_profile_budgets.argtypes = [pp, vp, vp, ctypes.c_int32, vp, vp, vp, vp]
        L.lukv_build_curves.argtypes = [pp, vp, vp, vp, vp]
        L.lukv_exact_workspace_bytes.argtypes = [pp, i64, ctypes.POINTER(sz)]
        L.lukv_exact_allocate.argtypes = [pp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.lukv_importance_workspace_bytes.argtypes = [pp, ctypes.c_int32, ctypes.POINTER(sz)]
        L.lukv_oracle_importance.argtypes = [pp, ctypes.c_int32, ctypes.c_int32, vp, vp, vp, vp, vp, ctypes.c_int32, vp,
                                             vp, sz, vp]
        L.lukv_score_ragged.argtypes = [pp, vp, vp, vp, vp, vp, sz, vp]
        L.lukv_score_keydiff.argtypes = [pp, vp, vp, vp, vp, sz, vp]
        L.lukv_compress_ragged.argtypes = [pp, vp] + L.lukv_compress.argtypes[1:]
        L.lukv_select_gather_ragged.argtypes = [pp, vp] + L.lukv_select_gather.argtypes[1:]
        L.lukv_profile_budgets_ragged.argtypes = [pp, vp] + L.lukv_profile_budgets.argtypes[1:]
        L.lukv_strerror.argtypes = [ctypes.c_int]
        L.lukv_strerror.restype = ctypes.c_char_p
        for name in EXPORTS[:5] + EXPORTS[6:]:
            getattr(L, name).restype = ctypes.c_int
        _lib = L
    return _lib


def strerror(code: int) -> str:
    return lib().lukv_strerror(int(code)).decode()


def make_params(S: int, L: int, H: int, G: int, d: int, T: int, w: int, kp: int, dtype, P: int,
                scale: float = 0.0, n_sink: int = 0, min_keep: float = 0.0, flags: int = 0) -> Params:
    if isinstance(dtype, torch.dtype):
        dtype = {torch.bfloat16: DTYPE_BF16, torch.float32: DTYPE_FP32}[dtype]
    elif isinstance(dtype, str):
        dtype = {"bf16": DTYPE_BF16, "fp32": DTYPE_FP32}[dtype]
    return Params(S, L, H, G, d, T, w, kp, int(dtype), P, float(scale), int(flags), int(n_sink), float(min_keep))


def _ptr(t) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        # without a device only argument validation can be exercised; it never launches
        return torch.cuda.current_stream().cuda_stream if torch.cuda.is_available() else 0
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _host_budgets(budgets_in: Sequence[int]) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(budgets_in, dtype=np.int64))


def lukv_workspace_bytes(params: Params) -> int:
    out = ctypes.c_size_t(0)
    rc = lib().lukv_workspace_bytes(ctypes.byref(params), ctypes.byref(out))
    if rc != OK:
        raise LukvError(rc, "lukv_workspace_bytes")
    return int(out.value)


def alloc_workspace(params: Params, device="cuda") -> torch.Tensor:
    """A device buffer of lukv_workspace_bytes() bytes (torch allocations are 256-byte aligned)."""
    return torch.empty(lukv_workspace_bytes(params), dtype=torch.uint8, device=device)


def _check(rc: int, where: str, check: bool) -> int:
    if check and rc != OK:
        raise LukvError(rc, where)
    return rc


def lukv_score(params: Params, q_win, k, scores, ws, stream=None, check: bool = True) -> int:
    rc = lib().lukv_score(ctypes.byref(params), _ptr(q_win), _ptr(k), _ptr(scores), _ptr(ws),
                          0 if ws is None else ws.numel() * ws.element_size(), _stream(stream))
    return _check(rc, "lukv_score", check)


def lukv_allocate(params: Params, curves, budgets_in, budgets, offsets, ws, stream=None, check: bool = True) -> int:
    b = _host_budgets(budgets_in)
    rc = lib().lukv_allocate(ctypes.byref(params), _ptr(curves), b.ctypes.data, _ptr(budgets), _ptr(offsets),
                             _ptr(ws), 0 if ws is None else ws.numel() * ws.element_size(), _stream(stream))
    return _check(rc, "lukv_allocate", check)


def lukv_allocate_static(params: Params, curves, budgets_in, budgets, offsets, stream=None, check: bool = True) -> int:
    """lukv_allocate without a workspace argument: the scratch is a fixed array inside the library
    (at most 262144 gains), for callers that cannot allocate device memory.  Calls sharing a device
    must not overlap on the GPU."""
    b = _host_budgets(budgets_in)
    rc = lib().lukv_allocate_static(ctypes.byref(params), _ptr(curves), b.ctypes.data, _ptr(budgets), _ptr(offsets),
                                    _stream(stream))
    return _check(rc, "lukv_allocate_static", check)


def _host_f32(x) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(x, dtype=np.float32).reshape(-1))


def lukv_profile_workspace_bytes(calib: Params, n_queries: int, n_ratios: int) -> int:
    out = ctypes.c_size_t(0)
    rc = lib().lukv_profile_workspace_bytes(ctypes.byref(calib), int(n_queries), int(n_ratios), ctypes.byref(out))
    if rc != OK:
        raise LukvError(rc, "lukv_profile_workspace_bytes")
    return int(out.value)


def lukv_profile_build(calib: Params, curves, n_queries: int, ratios, profile, ws, stream=None,
                       check: bool = True) -> int:
    """Offline profile: curves [n_queries][N][P] (device), ratios (host) -> profile [len(ratios)][N] (device)."""
    r = _host_f32(ratios)
    rc = lib().lukv_profile_build(ctypes.byref(calib), _ptr(curves), int(n_queries), r.ctypes.data, int(r.shape[0]),
                                  _ptr(profile), _ptr(ws), 0 if ws is None else ws.numel() * ws.element_size(),
                                  _stream(stream))
    return _check(rc, "lukv_profile_build", check)


def lukv_profile_budgets(params: Params, profile, ratios, sigma, budgets, offsets, stream=None,
                         check: bool = True) -> int:
    """Online lookup + budgeting: profile (device), ratios and per-sequence sigma (host) -> budgets, offsets."""
    r, sg = _host_f32(ratios), _host_f32(sigma)
    if sg.shape[0] != params.batch:
        raise ValueError("one target ratio per sequence")
    rc = lib().lukv_profile_budgets(ctypes.byref(params), _ptr(profile), r.ctypes.data, int(r.shape[0]),
                                    sg.ctypes.data, _ptr(budgets), _ptr(offsets), _stream(stream))
    return _check(rc, "lukv_profile_budgets", check)


def lukv_profile_budgets_ragged(params: Params, ctx_lens, profile, ratios, sigma, budgets, offsets, stream=None,
                                check: bool = True) -> int:
    """lukv_profile_budgets for sequences of different lengths: ctx_lens [S] host ints."""
    r, sg, lens = _host_f32(ratios), _host_f32(sigma), _host_lens(ctx_lens)
    if sg.shape[0] != params.batch:
        raise ValueError("one target ratio per sequence")
    rc = lib().lukv_profile_budgets_ragged(ctypes.byref(params), lens.ctypes.data, _ptr(profile), r.ctypes.data,
                                           int(r.shape[0]), sg.ctypes.data, _ptr(budgets), _ptr(offsets),
                                           _stream(stream))
    return _check(rc, "lukv_profile_budgets_ragged", check)


def lukv_build_curves(params: Params, scores, importance, curves, stream=None, check: bool = True) -> int:
    """Curves of the proxy ranking: scores, importance [S][N][n] -> curves [S][N][P] (all device)."""
    rc = lib().lukv_build_curves(ctypes.byref(params), _ptr(scores), _ptr(importance), _ptr(curves), _stream(stream))
    return _check(rc, "lukv_build_curves", check)


def lukv_importance_workspace_bytes(params: Params, k_max: int) -> int:
    out = ctypes.c_size_t(0)
    rc = lib().lukv_importance_workspace_bytes(ctypes.byref(params), int(k_max), ctypes.byref(out))
    if rc != OK:
        raise LukvError(rc, "lukv_importance_workspace_bytes")
    return int(out.value)


def lukv_oracle_importance(params: Params, k_max: int, d_model: int, q_dec, k, v, k_dec, w_o, normalize: bool,
                           importance, ws, stream=None, check: bool = True) -> int:
    """Oracle importance (Sec. 4.1): q_dec [S][L][H*G][k_max][d], k, v [S][L][H][T][d], k_dec [S][L][H][k_max][d] or
    None, w_o [L][H*G][d][d_model] -> importance [S][N][n] fp32 (all device)."""
    rc = lib().lukv_oracle_importance(ctypes.byref(params), int(k_max), int(d_model), _ptr(q_dec), _ptr(k), _ptr(v),
                                      _ptr(k_dec), _ptr(w_o), int(bool(normalize)), _ptr(importance), _ptr(ws),
                                      0 if ws is None else ws.numel() * ws.element_size(), _stream(stream))
    return _check(rc, "lukv_oracle_importance", check)


def lukv_exact_workspace_bytes(params: Params, max_budget: int) -> int:
    out = ctypes.c_size_t(0)
    rc = lib().lukv_exact_workspace_bytes(ctypes.byref(params), int(max_budget), ctypes.byref(out))
    if rc != OK:
        raise LukvError(rc, "lukv_exact_workspace_bytes")
    return int(out.value)


def lukv_exact_allocate(params: Params, curves, budgets_in, budgets, offsets, values, ws, stream=None,
                        check: bool = True) -> int:
    """Exact allocation on token-resolution curves; values is a float64 device tensor [S]."""
    b = _host_budgets(budgets_in)
    rc = lib().lukv_exact_allocate(ctypes.byref(params), _ptr(curves), b.ctypes.data, _ptr(budgets), _ptr(offsets),
                                   _ptr(values), _ptr(ws), 0 if ws is None else ws.numel() * ws.element_size(),
                                   _stream(stream))
    return _check(rc, "lukv_exact_allocate", check)


def lukv_select_gather(params: Params, scores, budgets, offsets, k, v, k_out, v_out, kept_idx, rows_cap: int, ws,
                       stream=None, check: bool = True) -> int:
    rc = lib().lukv_select_gather(ctypes.byref(params), _ptr(scores), _ptr(budgets), _ptr(offsets), _ptr(k), _ptr(v),
                                  _ptr(k_out), _ptr(v_out), _ptr(kept_idx), int(rows_cap), _ptr(ws),
                                  0 if ws is None else ws.numel() * ws.element_size(), _stream(stream))
    return _check(rc, "lukv_select_gather", check)


def lukv_select_gather_ragged(params: Params, ctx_lens, scores, budgets, offsets, k, v, k_out, v_out, kept_idx,
                              rows_cap: int, ws, stream=None, check: bool = True) -> int:
    """lukv_select_gather for sequences of different lengths: ctx_lens [S] host ints."""
    lens = _host_lens(ctx_lens)
    rc = lib().lukv_select_gather_ragged(ctypes.byref(params), lens.ctypes.data, _ptr(scores), _ptr(budgets),
                                         _ptr(offsets), _ptr(k), _ptr(v), _ptr(k_out), _ptr(v_out), _ptr(kept_idx),
                                         int(rows_cap), _ptr(ws), 0 if ws is None else ws.numel() * ws.element_size(),
                                         _stream(stream))
    return _check(rc, "lukv_select_gather_ragged", check)


def lukv_compress(params: Params, q_win, k, v, curves, budgets_in, k_out, v_out, kept_idx, budgets, offsets,
                  rows_cap: int, dev_status, ws, stream=None, check: bool = True) -> int:
    b = _host_budgets(budgets_in)
    rc = lib().lukv_compress(ctypes.byref(params), _ptr(q_win), _ptr(k), _ptr(v), _ptr(curves), b.ctypes.data,
                             _ptr(k_out), _ptr(v_out), _ptr(kept_idx), _ptr(budgets), _ptr(offsets), int(rows_cap),
                             _ptr(dev_status), _ptr(ws), 0 if ws is None else ws.numel() * ws.element_size(),
                             _stream(stream))
    return _check(rc, "lukv_compress", check)


def lukv_score_keydiff(params: Params, k, scores, ws, dev_status=None, stream=None, check: bool = True) -> int:
    """KeyDiff proxy scores: k [S][L][H][T][d] -> scores [S][N][n] fp32 (device); dev_status [1] int32 or None."""
    rc = lib().lukv_score_keydiff(ctypes.byref(params), _ptr(k), _ptr(scores), _ptr(dev_status), _ptr(ws),
                                  0 if ws is None else ws.numel() * ws.element_size(), _stream(stream))
    return _check(rc, "lukv_score_keydiff", check)


def _host_lens(ctx_lens) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(ctx_lens, dtype=np.int32))


def lukv_score_ragged(params: Params, ctx_lens, q_win, k, scores, ws, stream=None, check: bool = True) -> int:
    """lukv_score for sequences of different lengths: params.ctx_len is the row stride, ctx_lens [S] host ints."""
    lens = _host_lens(ctx_lens)
    rc = lib().lukv_score_ragged(ctypes.byref(params), lens.ctypes.data, _ptr(q_win), _ptr(k), _ptr(scores), _ptr(ws),
                                 0 if ws is None else ws.numel() * ws.element_size(), _stream(stream))
    return _check(rc, "lukv_score_ragged", check)


def lukv_compress_ragged(params: Params, ctx_lens, q_win, k, v, curves, budgets_in, k_out, v_out, kept_idx, budgets,
                         offsets, rows_cap: int, dev_status, ws, stream=None, check: bool = True) -> int:
    b = _host_budgets(budgets_in)
    lens = _host_lens(ctx_lens)
    rc = lib().lukv_compress_ragged(ctypes.byref(params), lens.ctypes.data, _ptr(q_win), _ptr(k), _ptr(v), _ptr(curves),
                                    b.ctypes.data, _ptr(k_out), _ptr(v_out), _ptr(kept_idx), _ptr(budgets),
                                    _ptr(offsets), int(rows_cap), _ptr(dev_status), _ptr(ws),
                                    0 if ws is None else ws.numel() * ws.element_size(), _stream(stream))
    return _check(rc, "lukv_compress_ragged", check)


def lukv_compress_profile(params: Params, q_win, k, v, curves, budgets_in, k_out, v_out, kept_idx, budgets, offsets,
                          rows_cap: int, dev_status, ws, stream=None, max_times: int = 64):
    """lukv_compress with a CUDA event after every kernel; synchronises.  Returns [(kernel name, ms)]."""
    b = _host_budgets(budgets_in)
    times = (KernelTime * max_times)()
    cnt = ctypes.c_int(0)
    rc = lib().lukv_compress_profile(ctypes.byref(params), _ptr(q_win), _ptr(k), _ptr(v), _ptr(curves), b.ctypes.data,
                                     _ptr(k_out), _ptr(v_out), _ptr(kept_idx), _ptr(budgets), _ptr(offsets),
                                     int(rows_cap), _ptr(dev_status), _ptr(ws),
                                     0 if ws is None else ws.numel() * ws.element_size(), _stream(stream), times,
                                     max_times, ctypes.byref(cnt))
    _check(rc, "lukv_compress_profile", True)
    return [(times[i].name.decode(), float(times[i].ms)) for i in range(cnt.value)]


def lukv_last_launch_count() -> int:
    return int(lib().lukv_last_launch_count())


class Outputs:
    """Caller-owned output buffers of one lukv_compress call, sized from the host-known row count."""

    def __init__(self, params: Params, budgets_in: Sequence[int], device="cuda", with_scores: bool = False):
        p = params
        self.rows = int(sum(int(b) for b in budgets_in)) + p.batch * p.N * p.window
        dt = torch.bfloat16 if p.dtype == DTYPE_BF16 else torch.float32
        self.k_out = torch.empty((self.rows, p.head_dim), dtype=dt, device=device)
        self.v_out = torch.empty((self.rows, p.head_dim), dtype=dt, device=device)
        self.kept_idx = torch.empty(self.rows, dtype=torch.int32, device=device)
        self.budgets = torch.empty((p.batch, p.N), dtype=torch.int32, device=device)
        self.offsets = torch.empty(p.batch * p.N + 1, dtype=torch.int32, device=device)
        self.dev_status = torch.zeros(1, dtype=torch.int32, device=device)
        self.scores = torch.empty((p.batch, p.N, p.n), dtype=torch.float32, device=device) if with_scores else None
