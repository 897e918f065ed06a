// Stages (c) and (d): per-head variable-k top-k selection and the packed gather.
//   select_kernel  one CTA per head: the b-th largest score is found by a bit-by-bit
//                  search over the order-preserving integer image of the scores
//                  (32 block-wide counts), then the kept positions are emitted in
//                  ascending order: everything above the threshold plus the first
//                  (lowest-position) ties.  This realises M^pi(b) of Sec. 3.2 / the
//                  "Eviction" step of Sec. 4.3 without a full sort.
//   gather_kernel  copies the kept K/V rows into the packed cache, 16 bytes per lane.
#include "common.cuh"

namespace lukv {
namespace {

constexpr int kSelThreads = 1024;

// Order-preserving map float -> uint32 (larger float <=> larger key).
__device__ __forceinline__ uint32_t score_key(float x) {
  const uint32_t b = __float_as_uint(x);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// Block-wide sum of one int per thread; every thread gets the result.  `buf` is one of
// two alternating shared arrays so that consecutive calls need a single barrier each.
__device__ __forceinline__ int block_sum(int v, int* buf) {
  v = __reduce_add_sync(0xffffffffu, v);
  if ((threadIdx.x & 31) == 0) buf[threadIdx.x >> 5] = v;
  __syncthreads();
  int total = 0;
#pragma unroll
  for (int i = 0; i < kSelThreads / 32; i += 4) {
    const int4 t = *reinterpret_cast<const int4*>(buf + i);
    total += t.x + t.y + t.z + t.w;
  }
  return total;
}

// EPT > 0: the thread keeps its EPT consecutive keys in registers (n <= 1024*EPT).
// EPT == 0: the thread re-reads its span of `per` consecutive scores from memory in every
// round (long contexts).
template <int EPT>
__global__ void __launch_bounds__(kSelThreads) select_kernel(const float* __restrict__ pooled,
                                                             const int32_t* __restrict__ budgets,
                                                             const int32_t* __restrict__ offsets,
                                                             int32_t* __restrict__ kept_idx, long long rows_cap, int n,
                                                             int w, int per) {
  __shared__ __align__(16) int cnt_buf[2][kSelThreads / 32];
  __shared__ int scan_gt[kSelThreads / 32], scan_eq[kSelThreads / 32];
  const int u = blockIdx.x, tid = threadIdx.x;
  const int b = budgets[u];
  const long long off = offsets[u];
  const float* src = pooled + (size_t)u * n;
  int32_t* out = kept_idx + off;
  const long long room = rows_cap - off;  // rows of this head that fit in the output

  // window rows follow the selected ones
  for (int t = tid; t < w; t += kSelThreads)
    if (b + t < room) out[b + t] = n + t;
  if (b <= 0) return;

  const int span = EPT > 0 ? EPT : per;
  const int j0 = tid * span;
  uint32_t keys[EPT > 0 ? EPT : 1];
  if (EPT > 0) {
#pragma unroll
    for (int e = 0; e < EPT; ++e) keys[e] = (j0 + e < n) ? score_key(src[j0 + e]) : 0u;
  }
  const int j_end = min(n, j0 + span);

  // b-th largest key: largest thr with count(key >= thr) >= b.  Positions beyond n carry
  // key 0 and are never counted because every candidate is non-zero.
  uint32_t thr = 0;
  int phase = 0;
  for (int bit = 31; bit >= 0; --bit) {
    const uint32_t cand = thr | (1u << bit);
    int c = 0;
    if (EPT > 0) {
#pragma unroll
      for (int e = 0; e < EPT; ++e) c += keys[e] >= cand;
    } else {
      for (int j = j0; j < j_end; ++j) c += score_key(src[j]) >= cand;
    }
    if (block_sum(c, cnt_buf[phase]) >= b) thr = cand;
    phase ^= 1;
  }

  // emit in ascending position: all keys > thr, and the first k_eq keys == thr
  int my_gt = 0, my_eq = 0;
  if (EPT > 0) {
#pragma unroll
    for (int e = 0; e < EPT; ++e) {
      my_gt += keys[e] > thr;
      my_eq += keys[e] == thr;
    }
  } else {
    for (int j = j0; j < j_end; ++j) {
      const uint32_t key = score_key(src[j]);
      my_gt += key > thr;
      my_eq += key == thr;
    }
  }
  // exclusive scans over the threads (thread order == position order)
  int inc_gt = my_gt, inc_eq = my_eq;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int a = __shfl_up_sync(0xffffffffu, inc_gt, o);
    const int c = __shfl_up_sync(0xffffffffu, inc_eq, o);
    if ((tid & 31) >= o) {
      inc_gt += a;
      inc_eq += c;
    }
  }
  if ((tid & 31) == 31) {
    scan_gt[tid >> 5] = inc_gt;
    scan_eq[tid >> 5] = inc_eq;
  }
  __syncthreads();
  int before_gt = inc_gt - my_gt, before_eq = inc_eq - my_eq, total_gt = 0;
  for (int wv = 0; wv < kSelThreads / 32; ++wv) {
    if (wv < (tid >> 5)) {
      before_gt += scan_gt[wv];
      before_eq += scan_eq[wv];
    }
    total_gt += scan_gt[wv];
  }
  const int k_eq = b - total_gt;  // ties to keep (>= 1)
  if (EPT > 0) {
#pragma unroll
    for (int e = 0; e < EPT; ++e) {
      const uint32_t key = keys[e];
      const bool gt = key > thr, eq = key == thr;
      if (gt || (eq && before_eq < k_eq)) {
        const int pos = before_gt + min(before_eq, k_eq);
        if (pos < room) out[pos] = j0 + e;
      }
      before_gt += gt;
      before_eq += eq;
    }
  } else {
    for (int j = j0; j < j_end; ++j) {
      const uint32_t key = score_key(src[j]);
      const bool gt = key > thr, eq = key == thr;
      if (gt || (eq && before_eq < k_eq)) {
        const int pos = before_gt + min(before_eq, k_eq);
        if (pos < room) out[pos] = j;
      }
      before_gt += gt;
      before_eq += eq;
    }
  }
}

// ---- gather --------------------------------------------------------------------------

constexpr int kGatherThreads = 256;

// LPR lanes copy one row of 16*LPR bytes.  A warp takes 32 consecutive packed rows: every
// lane resolves one row (source head by binary search over the offsets, source position
// from kept_idx), then the warp copies the rows 32/LPR at a time, four batches in flight.
template <int LPR>
__global__ void __launch_bounds__(kGatherThreads) gather_kernel(const int32_t* __restrict__ offsets,
                                                                const int32_t* __restrict__ kept_idx,
                                                                const uint4* __restrict__ k, const uint4* __restrict__ v,
                                                                uint4* __restrict__ k_out, uint4* __restrict__ v_out,
                                                                long long rows_cap, int heads, int T) {
  // rows actually present: the last offset, clipped to what the output can hold
  const long long total_rows = min((long long)__ldg(offsets + heads), rows_cap);
  constexpr int kRowsPerBatch = 32 / LPR;
  constexpr int kBatches = 32 / kRowsPerBatch;  // == LPR
  constexpr int kInFlight = LPR < 4 ? LPR : 4;
  const int lane = threadIdx.x & 31;
  const long long warp_global = ((long long)blockIdx.x * kGatherThreads + threadIdx.x) >> 5;
  const long long warps_total = ((long long)gridDim.x * kGatherThreads) >> 5;
  const int sub = lane / LPR, part = lane % LPR;
  for (long long base = warp_global * 32; base < total_rows; base += warps_total * 32) {
    const long long r = base + lane;
    long long src_row = -1;
    if (r < total_rows) {
      int lo = 0, hi = heads;  // largest u with offsets[u] <= r
      while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if ((long long)__ldg(offsets + mid) <= r) lo = mid; else hi = mid;
      }
      src_row = (long long)lo * T + __ldg(kept_idx + r);
    }
#pragma unroll
    for (int b0 = 0; b0 < kBatches; b0 += kInFlight) {
      uint4 kv[kInFlight], vv[kInFlight];
      long long srow[kInFlight];
#pragma unroll
      for (int i = 0; i < kInFlight; ++i) {
        const int row_in_span = (b0 + i) * kRowsPerBatch + sub;
        srow[i] = __shfl_sync(0xffffffffu, src_row, row_in_span);
        if (srow[i] >= 0) {
          kv[i] = __ldg(k + srow[i] * LPR + part);
          vv[i] = __ldg(v + srow[i] * LPR + part);
        }
      }
#pragma unroll
      for (int i = 0; i < kInFlight; ++i) {
        const int row_in_span = (b0 + i) * kRowsPerBatch + sub;
        if (srow[i] >= 0) {
          __stcs(k_out + (base + row_in_span) * LPR + part, kv[i]);
          __stcs(v_out + (base + row_in_span) * LPR + part, vv[i]);
        }
      }
    }
  }
}

template <int LPR>
void launch_gather_t(const Dims& dm, const int32_t* offsets, const int32_t* kept_idx, const void* k, const void* v,
                     void* k_out, void* v_out, long long rows_cap, cudaStream_t st) {
  const long long spans = (rows_cap + 31) / 32;
  long long blocks = (spans + kGatherThreads / 32 - 1) / (kGatherThreads / 32);
  const long long max_blocks = 148LL * 8 * 4;  // a few waves of resident CTAs; the loop covers the rest
  if (blocks > max_blocks) blocks = max_blocks;
  if (blocks < 1) blocks = 1;
  gather_kernel<LPR><<<(unsigned)blocks, kGatherThreads, 0, st>>>(offsets, kept_idx, (const uint4*)k, (const uint4*)v,
                                                                  (uint4*)k_out, (uint4*)v_out, rows_cap,
                                                                  (int)dm.heads(), dm.T);
}

}  // namespace

cudaError_t launch_select(const Dims& dm, const float* scores, bool scores_are_raw, const int32_t* budgets,
                          const int32_t* offsets, int32_t* kept_idx, int64_t rows_cap, LaunchCtx& lc) {
  cudaStream_t st = lc.st;
  (void)scores_are_raw;  // pooling is done by launch_pool before this call
  const unsigned grid = (unsigned)dm.heads();
  const int n = dm.n;
  if (n <= kSelThreads * 4)
    select_kernel<4><<<grid, kSelThreads, 0, st>>>(scores, budgets, offsets, kept_idx, rows_cap, n, dm.w, 4);
  else if (n <= kSelThreads * 16)
    select_kernel<16><<<grid, kSelThreads, 0, st>>>(scores, budgets, offsets, kept_idx, rows_cap, n, dm.w, 16);
  else if (n <= kSelThreads * 32)
    select_kernel<32><<<grid, kSelThreads, 0, st>>>(scores, budgets, offsets, kept_idx, rows_cap, n, dm.w, 32);
  else
    select_kernel<0><<<grid, kSelThreads, 0, st>>>(scores, budgets, offsets, kept_idx, rows_cap, n, dm.w,
                                                   (n + kSelThreads - 1) / kSelThreads);
  lc.mark("select");
  return cudaGetLastError();
}

cudaError_t launch_gather(const Dims& dm, const int32_t* offsets, const int32_t* kept_idx, const void* k,
                          const void* v, void* k_out, void* v_out, int64_t rows_cap, LaunchCtx& lc) {
  cudaStream_t st = lc.st;
  if (rows_cap <= 0) return cudaSuccess;
  const int lpr = (int)(dm.d * dm.esize() / 16);
  switch (lpr) {
    case 8: launch_gather_t<8>(dm, offsets, kept_idx, k, v, k_out, v_out, rows_cap, st); break;
    case 16: launch_gather_t<16>(dm, offsets, kept_idx, k, v, k_out, v_out, rows_cap, st); break;
    default: launch_gather_t<32>(dm, offsets, kept_idx, k, v, k_out, v_out, rows_cap, st); break;
  }
  lc.mark("gather");
  return cudaGetLastError();
}

}  // namespace lukv
