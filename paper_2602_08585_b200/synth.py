"""Seeded synthetic workloads for the LU-KV compression path.

This module only *draws inputs*; it contains none of the method's arithmetic and is the
one piece of code that both the CUDA path's callers and the CPU oracle's callers use.

Every tensor element is a pure function of (seed, tensor id, head index, element index):
a 32-bit counter hash picks one of 65 536 equiprobable quantiles of the target
distribution from a table built once on the host in float64.  Integer hashing and table
lookup are exact, so the same head can be drawn on the CPU (for the oracle) and on the GPU
(for the library) with identical bits, without copying multi-GB tensors around.

Workload shapes follow the five configurations of the benchmark definition: Llama-3.1-8B
like GQA shapes, long contexts of 1k..128k tokens, a few "massive" outlier channels in Q/K,
planted needle keys aligned with the observation-window queries, and non-concave
utility-versus-budget curves.  They stand in for the long-context evaluation workloads the
paper uses (needle-retrieval style contexts and long documents); no item of any such
suite is reproduced.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field, replace
from typing import Dict, List, Tuple

import numpy as np
import torch

_M32 = 0xFFFFFFFF
BASE_SEED = 20260208

# tensor ids
_TID_Q, _TID_K, _TID_V, _TID_NEEDLE_POS, _TID_NEEDLE_NOISE, _TID_OUTLIER, _TID_CURVE_E, _TID_CURVE_B = range(1, 9)
_TID_CALIB_HEAD, _TID_CALIB_E = 9, 10


@dataclass(frozen=True)
class Workload:
    name: str
    index: int            # configuration number (1-based); seed = BASE_SEED + index
    S: int                # sequences in the batch
    L: int                # layers
    H: int                # KV heads per layer
    G: int                # query heads per KV head
    d: int                # head dim
    T: int                # context length
    w: int                # observation window
    kp: int               # max-pool kernel
    dtype: str            # "bf16" | "fp32"
    P: int                # curve points per head
    keep: Tuple[float, ...]   # kept fraction per sequence (cycled over the batch)
    needles: int          # planted needle keys per head
    outlier_channels: int = 4
    outlier_kind: str = "x8"  # "none" | "x8" | "student_t3" (K only; Q keeps x8)

    @property
    def N(self) -> int:
        return self.L * self.H

    @property
    def n(self) -> int:
        return self.T - self.w

    @property
    def seed(self) -> int:
        return BASE_SEED + self.index

    @property
    def torch_dtype(self):
        return torch.bfloat16 if self.dtype == "bf16" else torch.float32

    def budgets(self) -> np.ndarray:
        """Selectable tokens per sequence: floor(keep * N * T); window rows are kept on top."""
        return np.array([int(math.floor(self.keep[q % len(self.keep)] * self.N * self.T)) for q in range(self.S)],
                        dtype=np.int64)

    def total_rows(self) -> int:
        return int(self.budgets().sum()) + self.S * self.N * self.w


CONFIGS: Dict[str, Workload] = {
    "tiny": Workload("tiny", 1, S=1, L=1, H=4, G=1, d=64, T=1024, w=16, kp=7, dtype="fp32", P=65,
                     keep=(0.2,), needles=8, outlier_channels=0, outlier_kind="none"),
    "llama8b_1layer_8k": Workload("llama8b_1layer_8k", 2, S=1, L=1, H=8, G=4, d=128, T=8192, w=32, kp=7,
                                  dtype="bf16", P=129, keep=(0.2,), needles=64),
    "llama8b_32k": Workload("llama8b_32k", 3, S=1, L=32, H=8, G=4, d=128, T=32768, w=32, kp=7, dtype="bf16",
                            P=257, keep=(0.2,), needles=64),
    "batch8_16k_mixed": Workload("batch8_16k_mixed", 4, S=8, L=32, H=8, G=4, d=128, T=16384, w=64, kp=5,
                                 dtype="bf16", P=257, keep=(0.1, 0.5), needles=64),
    "gqa7_128k": Workload("gqa7_128k", 5, S=1, L=28, H=4, G=7, d=128, T=131072, w=32, kp=7, dtype="bf16",
                          P=513, keep=(0.1,), needles=256, outlier_kind="student_t3"),
}


def scaled(wl: Workload, **kw) -> Workload:
    """A copy of a workload with some sizes changed (used for reduced parity cases)."""
    return replace(wl, **kw)


# ---- counter hash ------------------------------------------------------------------------

def _mix32_int(x: int) -> int:
    x &= _M32
    x ^= x >> 16
    x = (x * 0x7FEB352D) & _M32
    x ^= x >> 15
    x = (x * 0x846CA68B) & _M32
    x ^= x >> 16
    return x


def _mul32(x: torch.Tensor, c: int) -> torch.Tensor:
    """(x * c) mod 2^32 for int64 tensors holding values < 2^32, without int64 overflow."""
    lo = (x & 0xFFFF) * c
    hi = (((x >> 16) * c) & 0xFFFF) << 16
    return (lo + hi) & _M32


def _mix32(x: torch.Tensor) -> torch.Tensor:
    x = x ^ (x >> 16)
    x = _mul32(x, 0x7FEB352D)
    x = x ^ (x >> 15)
    x = _mul32(x, 0x846CA68B)
    x = x ^ (x >> 16)
    return x


def _stream_key(seed: int, tid: int, u: int) -> Tuple[int, int]:
    k1 = _mix32_int(seed ^ _mix32_int(tid * 0x9E3779B9 + 0x85EBCA6B))
    k1 = _mix32_int(k1 ^ _mix32_int(u + 0xC2B2AE35))
    k2 = _mix32_int(k1 + 0x27D4EB2F)
    return k1, k2


def _hash_u32(seed: int, tid: int, u: int, count: int, device) -> torch.Tensor:
    """count 32-bit hashes (int64 tensor, values < 2^32) for stream (seed, tid, u)."""
    k1, k2 = _stream_key(seed, tid, u)
    e = torch.arange(count, dtype=torch.int64, device=device)
    return _mix32((_mix32(e ^ k1) + k2) & _M32)


def _hash_u32_host(seed: int, tid: int, u: int, count: int) -> np.ndarray:
    return _hash_u32(seed, tid, u, count, "cpu").numpy()


# ---- quantile tables ---------------------------------------------------------------------

_TABLES: Dict[Tuple[str, str], torch.Tensor] = {}


def _table(kind: str, device) -> torch.Tensor:
    key = (kind, str(device))
    if key not in _TABLES:
        hkey = (kind, "cpu")
        if hkey not in _TABLES:
            from scipy import special, stats
            p = (np.arange(65536, dtype=np.float64) + 0.5) / 65536.0
            vals = special.ndtri(p) if kind == "normal" else stats.t.ppf(p, 3)
            _TABLES[hkey] = torch.from_numpy(vals.astype(np.float32))
        _TABLES[key] = _TABLES[hkey].to(device)
    return _TABLES[key]


def _draw(kind: str, seed: int, tid: int, u: int, count: int, device) -> torch.Tensor:
    h = _hash_u32(seed, tid, u, count, device)
    return _table(kind, device)[h >> 16]


# ---- per-head tensors --------------------------------------------------------------------

def head_index(wl: Workload, q: int, layer: int, h: int) -> int:
    return (q * wl.L + layer) * wl.H + h


def outlier_channels(wl: Workload, u: int) -> List[int]:
    """The head's outlier channel ids (shared by K and by the G query heads of the KV head)."""
    if wl.outlier_kind == "none" or wl.outlier_channels == 0:
        return []
    hs = _hash_u32_host(wl.seed, _TID_OUTLIER, u, 64)
    chans: List[int] = []
    for v in hs:
        c = int(v) % wl.d
        if c not in chans:
            chans.append(c)
        if len(chans) == wl.outlier_channels:
            break
    return chans


def needle_positions(wl: Workload, u: int) -> List[int]:
    hs = _hash_u32_host(wl.seed, _TID_NEEDLE_POS, u, 4 * wl.needles + 64)
    pos: List[int] = []
    seen = set()
    for v in hs:
        p = int(v) % wl.n
        if p not in seen:
            seen.add(p)
            pos.append(p)
        if len(pos) == wl.needles:
            break
    return pos


def _q_head_f32(wl: Workload, u: int, device) -> torch.Tensor:
    z = _draw("normal", wl.seed, _TID_Q, u, wl.G * wl.w * wl.d, device).view(wl.G, wl.w, wl.d)
    ch = outlier_channels(wl, u)
    if ch:
        z = z.clone()
        z[:, :, ch] *= 8.0
    return z


def gen_head(wl: Workload, q: int, layer: int, h: int, device="cpu"):
    """(q_head [G][w][d], k_head [T][d], v_head [T][d]) of one KV head, in the workload's dtype."""
    u = head_index(wl, q, layer, h)
    dt = wl.torch_dtype
    ch = outlier_channels(wl, u)
    q_head = _q_head_f32(wl, u, device).to(dt)
    k = _draw("normal", wl.seed, _TID_K, u, wl.T * wl.d, device).view(wl.T, wl.d)
    if ch:
        k = k.clone()
        if wl.outlier_kind == "student_t3":
            t = _draw("student_t3", wl.seed, _TID_OUTLIER + 100, u, wl.T * len(ch), device).view(wl.T, len(ch))
            k[:, ch] = t
        else:
            k[:, ch] *= 8.0
    k_head = k.to(dt)
    v_head = _draw("normal", wl.seed, _TID_V, u, wl.T * wl.d, device).view(wl.T, wl.d).to(dt)
    # needles: 3 x (mean of the rounded window queries) + N(0, 0.1^2) noise, computed on the
    # host in float64 so that every device plants identical rows
    if wl.needles > 0:
        q_cpu = _q_head_f32(wl, u, "cpu").to(dt).to(torch.float64)
        m = q_cpu.reshape(-1, wl.d).mean(dim=0)
        pos = needle_positions(wl, u)
        z = _draw("normal", wl.seed, _TID_NEEDLE_NOISE, u, len(pos) * wl.d, "cpu").view(len(pos), wl.d)
        rows = (3.0 * m[None, :] + 0.1 * z.to(torch.float64)).to(torch.float32).to(dt)
        k_head[torch.tensor(pos, dtype=torch.int64, device=k_head.device)] = rows.to(k_head.device)
    return q_head, k_head, v_head


def gen_tensors(wl: Workload, device="cpu"):
    """Full tensors: q [S][L][H*G][w][d], k/v [S][L][H][T][d]."""
    dt = wl.torch_dtype
    qt = torch.empty((wl.S, wl.L, wl.H * wl.G, wl.w, wl.d), dtype=dt, device=device)
    kt = torch.empty((wl.S, wl.L, wl.H, wl.T, wl.d), dtype=dt, device=device)
    vt = torch.empty((wl.S, wl.L, wl.H, wl.T, wl.d), dtype=dt, device=device)
    for q in range(wl.S):
        for layer in range(wl.L):
            for h in range(wl.H):
                qh, kh, vh = gen_head(wl, q, layer, h, device)
                qt[q, layer, h * wl.G:(h + 1) * wl.G] = qh
                kt[q, layer, h] = kh
                vt[q, layer, h] = vh
    return qt, kt, vt


def gen_curves(wl: Workload, concave: bool = False) -> np.ndarray:
    """Utility-versus-budget curves [N][P] float32, shared by all sequences of the batch.

    Point k is the utility of keeping the top k*T/(P-1) non-window tokens.  Increments are
    Exp(1) draws, one in five scaled x3 (which makes the curve non-concave).  With
    ``concave=True`` the same increments are sorted in decreasing order per head.
    """
    out = np.zeros((wl.N, wl.P), dtype=np.float32)
    for hid in range(wl.N):
        he = _hash_u32_host(wl.seed, _TID_CURVE_E, hid, wl.P - 1).astype(np.float64)
        hb = _hash_u32_host(wl.seed, _TID_CURVE_B, hid, wl.P - 1).astype(np.float64)
        uexp = (he + 0.5) / 4294967296.0
        inc = -np.log1p(-uexp)
        inc = inc * np.where(hb / 4294967296.0 < 0.2, 3.0, 1.0)
        if concave:
            inc = np.sort(inc)[::-1]
        out[hid, 1:] = np.cumsum(inc).astype(np.float32)
    return out


def gen_calibration_curves(seed: int, n_queries: int, N: int, T: int) -> np.ndarray:
    """Token-resolution utility curves [n_queries][N][T+1] float32 of a calibration context of T tokens,
    one set per calibration query (the inputs of the offline profile; the paper's default
    calibration set is a context of about 4,000 tokens with 30 queries).

    Each head has a decay exponent in [0.2, 1.6] and a scale in [0.25, 4] that all queries
    share, which gives the heads the consistent preference across queries that the profile
    averages over; the increment of token k is scale * (k+1)^-exponent times an Exp(1) draw
    per (query, head, token), so single curves are noisy and non-concave.
    """
    out = np.zeros((n_queries, N, T + 1), dtype=np.float32)
    k = np.arange(1, T + 1, dtype=np.float64)
    for hid in range(N):
        hh = _hash_u32_host(seed, _TID_CALIB_HEAD, hid, 2).astype(np.float64) / 4294967296.0
        alpha = 0.2 + 1.4 * hh[0]
        scale = 0.25 * 16.0 ** hh[1]
        trend = scale * k ** (-alpha)
        for i in range(n_queries):
            he = _hash_u32_host(seed, _TID_CALIB_E, i * N + hid, T).astype(np.float64)
            inc = -np.log1p(-(he + 0.5) / 4294967296.0) * trend
            out[i, hid, 1:] = np.cumsum(inc).astype(np.float32)
    return out


def to_numpy_bits(t: torch.Tensor) -> np.ndarray:
    """A CPU numpy view of a tensor for the oracle: bf16 -> uint16 bit patterns, fp32 as is."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()
