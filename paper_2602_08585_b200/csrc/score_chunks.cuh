// The per-chunk arithmetic of the two-sweep tensor-core scorer (32 accumulator columns of one TMEM lane at a
// time), shared with the epilogue micro-benchmark so that it times exactly the code the kernel runs.
#pragma once
#include "tc_ptx.cuh"

namespace lukv {
namespace {

// Pass 1, 32 columns (keys jbase..jbase+31) of one query row: fold into the running (m, l).
// (m, l) means sum over the keys seen so far of exp2(x - m); m is a reference point, not
// necessarily the maximum: the common path adds the new terms relative to the current m and
// only re-references (exactly, from the chunk maximum) when the chunk sum leaves a safe range
// -- which also covers the first chunk (m = -inf) and any overflow.
template <bool MASKED>
__device__ __forceinline__ void p1_chunk(const float (&v)[32], int jbase, int lim, float scale_log2, float& m,
                                         float& l) {
  float x[32];
#pragma unroll
  for (int i = 0; i < 32; ++i) x[i] = (!MASKED || jbase + i <= lim) ? v[i] : -INFINITY;
  const uint64_t sc2 = pack2(scale_log2, scale_log2), nm2 = pack2(-m, -m);
  uint64_t acc0 = 0ull, acc1 = 0ull;  // bit pattern of (+0, +0)
  // The polynomial has no overflow of its own (its exponent arithmetic wraps), so the largest argument that
  // goes through it is checked once per chunk instead: it joins the test that sends the chunk to the exact path.
  float pmax = -INFINITY;
#pragma unroll
  for (int i = 0; i < 32; i += 4) {
    acc0 = fadd2(acc0, ex2_pair(ffma2(pack2(x[i], x[i + 1]), sc2, nm2)));
    if (LUKV_POLY_SEL1(i)) {
      pmax = fmaxf(pmax, fmaxf(x[i + 2], x[i + 3]));
      acc1 = fadd2(acc1, ex2_poly_pair<false>(ffma2(pack2(x[i + 2], x[i + 3]), sc2, nm2)));
    } else {
      acc1 = fadd2(acc1, ex2_pair(ffma2(pack2(x[i + 2], x[i + 3]), sc2, nm2)));
    }
  }
  const float cs = sum4(acc0, acc1);
  if (cs <= 1e12f && fmaf(pmax, scale_log2, -m) <= 100.f) {  // false for inf and NaN
    l += cs;
    return;
  }
  float cmax = x[0];
#pragma unroll
  for (int i = 1; i < 32; ++i) cmax = fmaxf(cmax, x[i]);
  if (cmax == -INFINITY) return;  // every key of the chunk is masked
  const float mn = fmaxf(m, cmax * scale_log2);  // scale > 0
  float a0 = l * ex2(m - mn), a1 = 0.f;
#pragma unroll
  for (int i = 0; i < 32; i += 2) {
    a0 += ex2(fmaf(x[i], scale_log2, -mn));
    a1 += ex2(fmaf(x[i + 1], scale_log2, -mn));
  }
  l = a0 + a1;
  m = mn;
}

// Pass 2, 32 columns (query rows c0..c0+31) of one key: add the probabilities.  The -lse of the rows is read from
// shared memory.
__device__ __forceinline__ void p2_chunk(const float (&v)[32], const float* nlse, uint64_t sc2, uint64_t& acc0,
                                         uint64_t& acc1) {
#pragma unroll
  for (int i = 0; i < 32; i += 4) {
    const ulonglong2 ls = *reinterpret_cast<const ulonglong2*>(nlse + i);  // (-lse[i], -lse[i+1]), (-lse[i+2], -lse[i+3])
    acc0 = fadd2(acc0, ex2_pair(ffma2(pack2(v[i], v[i + 1]), sc2, ls.x)));
    if (LUKV_POLY_SEL2(i)) acc1 = fadd2(acc1, ex2_poly_pair<false>(ffma2(pack2(v[i + 2], v[i + 3]), sc2, ls.y)));
    else acc1 = fadd2(acc1, ex2_pair(ffma2(pack2(v[i + 2], v[i + 3]), sc2, ls.y)));
  }
}

// Variant for the micro-benchmark's comparison: the -lse values come out of registers (lane l of the warp holds
// rows 4l..4l+3 of a block of 128 rows in `mine`; every lane fetches the four it needs next by shuffles; c0 is a
// multiple of 32 below 128).  With the tensor pipe streaming operands out of shared memory all the time this is
// much faster in isolation (1111 against 1810 clocks per tile), but inside the scorer, where the pipe is busy
// under half of the time and the shuffles cost issue slots, it was slower (0.827 against 0.797 ms).
__device__ __forceinline__ void p2_chunk_shfl(const float (&v)[32], const float4 mine, int c0, uint64_t sc2, uint64_t& acc0,
                                              uint64_t& acc1) {
#pragma unroll
  for (int i = 0; i < 32; i += 4) {
    const int src = (c0 + i) >> 2;
    const float l0 = __shfl_sync(0xffffffffu, mine.x, src), l1 = __shfl_sync(0xffffffffu, mine.y, src);
    const float l2 = __shfl_sync(0xffffffffu, mine.z, src), l3 = __shfl_sync(0xffffffffu, mine.w, src);
    acc0 = fadd2(acc0, ex2_pair(ffma2(pack2(v[i], v[i + 1]), sc2, pack2(l0, l1))));
    if (LUKV_POLY_SEL2(i)) acc1 = fadd2(acc1, ex2_poly_pair<false>(ffma2(pack2(v[i + 2], v[i + 3]), sc2, pack2(l2, l3))));
    else acc1 = fadd2(acc1, ex2_pair(ffma2(pack2(v[i + 2], v[i + 3]), sc2, pack2(l2, l3))));
  }
}

}  // namespace
}  // namespace lukv
