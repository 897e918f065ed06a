// Stages (c) and (d): per-head variable-k top-k selection and the packed gather.
//   select_kernel  one CTA per head, or a thread-block cluster of 2, 4 or 8 CTAs per head that merge their
//                  histograms and counts through distributed shared memory (long contexts; few heads):
//                  the b-th largest score is found digit by digit (11, 11
//                  and 10 bits) over the order-preserving integer image of the scores, each
//                  digit from a shared-memory histogram, then the kept positions are emitted in
//                  ascending order: everything above the threshold plus the first
//                  (lowest-position) ties.  This realises M^pi(b) of Sec. 3.2 / the
//                  "Eviction" step of Sec. 4.3 without a full sort.
//   gather_kernel  copies the kept K/V rows into the packed cache, 16 bytes per lane.
#include <cooperative_groups.h>

#include "common.cuh"

namespace lukv {
namespace {

namespace cg = cooperative_groups;

constexpr int kSelThreads = 1024;
constexpr int kSelWarps = kSelThreads / 32;

// Order-preserving map float -> uint32 (larger float <=> larger key).
__device__ __forceinline__ uint32_t score_key(float x) {
  const uint32_t b = __float_as_uint(x);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// Key of position j: attention sinks (the first n_sink positions, App. E) get the largest key, so
// they rank before every scored position; among themselves the lower position wins like any tie.
__device__ __forceinline__ uint32_t key_at(const float* src, int j, int n_sink) {
  return j < n_sink ? 0xFFFFFFFFu : score_key(src[j]);
}

// One CTA per head (CLUSTER false) or one cluster of CTAs per head (CLUSTER true; CTA r of the cluster owns the
// positions [r*32*span, (r+1)*32*span)).  Warp wv of a CTA owns span consecutive positions and lane l of it the
// positions e*32 + l of those, so loads are coalesced and position order is (CTA, warp, e, lane).
// EPT > 0: span = 32*EPT and the thread keeps its EPT keys in registers (n <= 1024*EPT).
// EPT == 0: span is a multiple of 32 given by the host and the keys are re-read from memory
// in every round (long contexts).
template <int EPT, bool CLUSTER>
__global__ void __launch_bounds__(kSelThreads, 1) select_kernel(const float* __restrict__ pooled,
                                                                const int32_t* __restrict__ budgets,
                                                                const int32_t* __restrict__ offsets,
                                                                int32_t* __restrict__ kept_idx, long long rows_cap,
                                                                int n_stride, int w, int span_rt, int head0, int n_sink,
                                                                SeqLens sl, int heads_per_seq) {
  __shared__ int hist[2048];
  __shared__ int scan_gt[kSelWarps], scan_eq[kSelWarps];
  __shared__ int sel_digit, sel_want;
  __shared__ int cta_tot[2];  // keys of this CTA above / equal to the threshold
  static_assert(!CLUSTER || EPT > 0, "a cluster keeps its keys in registers");
  cg::cluster_group cluster = cg::this_cluster();
  const int csize = CLUSTER ? (int)cluster.num_blocks() : 1, crank = CLUSTER ? (int)cluster.block_rank() : 0;
  const int u = head0 + (int)blockIdx.x / csize, tid = threadIdx.x, lane = tid & 31, wv = tid >> 5;
  const int b = budgets[u];
  const long long off = offsets[u];
  // n_stride: row stride of the scores (the longest sequence); n: rankable positions of this head's sequence
  const int n = heads_per_seq > 0 ? sl.T[u / heads_per_seq] - w : n_stride;
  const float* src = pooled + (size_t)u * n_stride;
  int32_t* out = kept_idx + off;
  const long long room = rows_cap - off;  // rows of this head that fit in the output

  // window rows follow the selected ones
  if (crank == 0)
    for (int t = tid; t < w; t += kSelThreads)
      if (b + t < room) out[b + t] = n + t;
  if (b <= 0) return;  // the whole cluster leaves

  const int span = EPT > 0 ? 32 * EPT : span_rt;
  const int base = (crank * kSelWarps + wv) * span + lane;
  const int iters = span >> 5;
  uint32_t keys[EPT > 0 ? EPT : 1];
  if (EPT > 0) {
#pragma unroll
    for (int e = 0; e < EPT; ++e) {
      const int j = base + 32 * e;
      keys[e] = j < n ? score_key(src[j]) : 0u;
    }
    if (base - lane < n_sink) {  // only the warps whose span starts below n_sink hold sink positions
#pragma unroll
      for (int e = 0; e < EPT; ++e)
        if (base + 32 * e < n_sink) keys[e] = 0xFFFFFFFFu;
    }
  }

  // b-th largest key: the largest thr with count(key >= thr) >= b, found digit by digit (11, 11 and
  // 10 bits, most significant first): the keys that match the digits fixed so far are counted into
  // a shared-memory histogram of the next digit, and the bin in which the count of larger keys
  // reaches the remaining budget is the next digit of thr.  Positions beyond n take no part.
  uint32_t thr = 0;
  {
    int want = b;  // keys still to be found among those that match the fixed digits
#pragma unroll 1
    for (int pass = 0; pass < 3; ++pass) {
      const int shift = pass == 0 ? 21 : (pass == 1 ? 10 : 0);
      const int bins = pass == 2 ? 1024 : 2048;
      const uint32_t above = pass == 0 ? 0u : (thr >> (shift + (pass == 1 ? 11 : 10)));  // the fixed digits
      for (int i = tid; i < bins; i += kSelThreads) hist[i] = 0;
      __syncthreads();
      auto count = [&](uint32_t key, int j) {
        if (j < n && (pass == 0 || (key >> (shift + (pass == 1 ? 11 : 10))) == above))
          atomicAdd(&hist[(key >> shift) & (uint32_t)(bins - 1)], 1);
      };
      if (EPT > 0) {
#pragma unroll
        for (int e = 0; e < EPT; ++e) count(keys[e], base + 32 * e);
      } else {
        for (int e = 0; e < iters; ++e) {
          const int j = base + 32 * e;
          count(j < n ? key_at(src, j, n_sink) : 0u, j);
        }
      }
      if (CLUSTER) cluster.sync(); else __syncthreads();  // every histogram of the head is complete
      // thread t owns the bins [t*per, t*per+per); suffix sums over the threads, from the top
      const int per = bins / kSelThreads;  // 2 or 1
      // the bins of this thread, added over the CTAs of the head (every CTA computes the same)
      int merged0 = 0, merged1 = 0;
      if (CLUSTER) {
        for (int c = 0; c < csize; ++c) {
          const int* remote = cluster.map_shared_rank(hist, c) + tid * per;
          merged0 += remote[0];
          if (per == 2) merged1 += remote[1];
        }
      } else {
        merged0 = hist[tid * per];
        if (per == 2) merged1 = hist[tid * per + 1];
      }
      const int mine = merged0 + merged1;
      int incl = mine;  // sum over the lanes >= this one
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const int o = __shfl_down_sync(0xffffffffu, incl, off);
        if (lane + off < 32) incl += o;
      }
      if (lane == 0) scan_gt[wv] = incl;  // warp totals (scan_gt is free until the emit phase)
      __syncthreads();
      int higher = 0;  // keys in bins above this thread's bins
      for (int x = wv + 1; x < kSelWarps; ++x) higher += scan_gt[x];
      higher += incl - mine;
      if (higher < want && want <= higher + mine) {  // exactly one thread: the digit is in its bins
        int run = higher;
        for (int i = per - 1; i >= 0; --i) {
          const int c = i ? merged1 : merged0;
          if (want <= run + c) {
            sel_digit = tid * per + i;
            sel_want = want - run;
            break;
          }
          run += c;
        }
      }
      if (CLUSTER) cluster.sync(); else __syncthreads();  // the histograms may be cleared again
      thr |= (uint32_t)sel_digit << shift;
      want = sel_want;
    }
  }

  // per-warp totals of keys above / equal to the threshold, then an exclusive scan over warps
  int my_gt = 0, my_eq = 0;
  if (EPT > 0) {
#pragma unroll
    for (int e = 0; e < EPT; ++e) {
      my_gt += keys[e] > thr;
      my_eq += keys[e] == thr;
    }
  } else {
    for (int e = 0; e < iters; ++e) {
      const int j = base + 32 * e;
      const uint32_t key = j < n ? key_at(src, j, n_sink) : 0u;
      my_gt += key > thr;
      my_eq += key == thr;
    }
  }
  my_gt = __reduce_add_sync(0xffffffffu, my_gt);
  my_eq = __reduce_add_sync(0xffffffffu, my_eq);
  if (lane == 0) {
    scan_gt[wv] = my_gt;
    scan_eq[wv] = my_eq;
  }
  __syncthreads();
  int run_gt = 0, run_eq = 0, total_gt = 0;
  for (int x = 0; x < kSelWarps; ++x) {
    if (x < wv) {
      run_gt += scan_gt[x];
      run_eq += scan_eq[x];
    }
    total_gt += scan_gt[x];
  }
  if (CLUSTER) {
    // the CTAs before this one along the positions come first; the totals run over the whole head
    if (tid == 0) {
      int eq = 0;
      for (int x = 0; x < kSelWarps; ++x) eq += scan_eq[x];
      cta_tot[0] = total_gt;
      cta_tot[1] = eq;
    }
    cluster.sync();
    total_gt = 0;
    for (int c = 0; c < csize; ++c) {
      const int* tot = cluster.map_shared_rank(cta_tot, c);
      const int g = tot[0], q = tot[1];
      if (c < crank) {
        run_gt += g;
        run_eq += q;
      }
      total_gt += g;
    }
    cluster.sync();  // no CTA of the cluster exits while another may still read its shared memory
  }
  const int k_eq = b - total_gt;  // ties to keep (>= 1)

  // emit in ascending position: all keys > thr, and the first k_eq keys == thr
  const uint32_t lt_mask = (1u << lane) - 1u;
  auto emit = [&](uint32_t key, int j) {
    const bool gt = key > thr, eq = key == thr;
    const uint32_t m_gt = __ballot_sync(0xffffffffu, gt), m_eq = __ballot_sync(0xffffffffu, eq);
    const int before_gt = run_gt + __popc(m_gt & lt_mask);
    const int before_eq = run_eq + __popc(m_eq & lt_mask);
    if (gt || (eq && before_eq < k_eq)) {
      const int pos = before_gt + min(before_eq, k_eq);
      if (pos < room) out[pos] = j;
    }
    run_gt += __popc(m_gt);
    run_eq += __popc(m_eq);
  };
  if (EPT > 0) {
#pragma unroll
    for (int e = 0; e < EPT; ++e) emit(keys[e], base + 32 * e);
  } else {
    for (int e = 0; e < iters; ++e) {
      const int j = base + 32 * e;
      emit(j < n ? key_at(src, j, n_sink) : 0u, j);
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
                                                                long long rows_cap, int head0, int nheads, int T) {
  // packed rows of heads [head0, head0+nheads), clipped to what the output can hold
  const long long row_begin = __ldg(offsets + head0);
  const long long total_rows = min((long long)__ldg(offsets + head0 + nheads), rows_cap);
  constexpr int kRowsPerBatch = 32 / LPR;
  constexpr int kBatches = 32 / kRowsPerBatch;  // == LPR
  constexpr int kInFlight = LPR < 4 ? LPR : 4;
  const int lane = threadIdx.x & 31;
  const long long warp_global = ((long long)blockIdx.x * kGatherThreads + threadIdx.x) >> 5;
  const long long warps_total = ((long long)gridDim.x * kGatherThreads) >> 5;
  const int sub = lane / LPR, part = lane % LPR;
  for (long long base = row_begin + warp_global * 32; base < total_rows; base += warps_total * 32) {
    const long long r = base + lane;
    long long src_row = -1;
    if (r < total_rows) {
      int lo = head0, hi = head0 + nheads;  // largest u with offsets[u] <= r
      while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if ((long long)__ldg(offsets + mid) <= r) lo = mid; else hi = mid;
      }
      // positions come from the selection kernel; clamping them keeps the copy inside the head even if
      // the scores were not finite (their ranking is then meaningless, but nothing is read out of bounds)
      const int pos = min(max(__ldg(kept_idx + r), 0), T - 1);
      src_row = (long long)lo * T + pos;
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
                     void* k_out, void* v_out, long long rows_cap, HeadRange hr, cudaStream_t st) {
  // the rows of a head range are only known on the device; size the grid for its share of the output
  // (a capacity beyond what the call can ever produce sizes nothing: clamp it first)
  const long long rows_max = (long long)dm.heads() * dm.T;
  if (rows_cap > rows_max) rows_cap = rows_max;
  const long long spans = (rows_cap * hr.nh / (long long)dm.heads() + 31) / 32 + 1;
  long long blocks = (spans + kGatherThreads / 32 - 1) / (kGatherThreads / 32);
  const long long max_blocks = 148LL * 8 * 4;  // a few waves of resident CTAs; the loop covers the rest
  if (blocks > max_blocks) blocks = max_blocks;
  if (blocks < 1) blocks = 1;
  gather_kernel<LPR><<<(unsigned)blocks, kGatherThreads, 0, st>>>(offsets, kept_idx, (const uint4*)k, (const uint4*)v,
                                                                  (uint4*)k_out, (uint4*)v_out, rows_cap, hr.h0,
                                                                  hr.nh, dm.T);
}

}  // namespace

cudaError_t launch_select(const Dims& dm, const float* scores, const int32_t* budgets, const int32_t* offsets,
                          int32_t* kept_idx, int64_t rows_cap, HeadRange hr, LaunchCtx& lc) {
  cudaStream_t st = lc.st;
  const unsigned grid = (unsigned)hr.nh;
  const int n = dm.n;
  SeqLens sl = {};
  const int hps = dm.seq_T ? dm.N : 0;
  if (dm.seq_T)
    for (int q = 0; q < dm.S; ++q) sl.T[q] = dm.seq_T[q];
  // Keys per thread (in registers) and CTAs per head.  Up to 32768 positions: one CTA with 2, 8, 16 or 32 keys per
  // thread (a cluster's barriers cost more than they save there).  Up to 262144: the smallest cluster (2, 4 or 8
  // CTAs) that covers the head with 32 keys per thread; small clusters are placed and synchronised faster than large
  // ones.  Beyond: one CTA that re-reads its keys from memory in every round.
  int ept = 0, csize = 1;
  if (n <= kSelThreads * 32) {
    ept = n <= kSelThreads * 2 ? 2 : n <= kSelThreads * 8 ? 8 : n <= kSelThreads * 16 ? 16 : 32;
  } else {
    for (int c : {2, 4, 8})
      if (!ept && (long long)c * kSelThreads * 32 >= n) ept = 32, csize = c;
  }
  if (ept == 0) {
    const int per_warp = (n + kSelWarps - 1) / kSelWarps;
    const int span = (per_warp + 31) & ~31;
    select_kernel<0, false><<<grid, kSelThreads, 0, st>>>(scores, budgets, offsets, kept_idx, rows_cap, n, dm.w, span,
                                                          hr.h0, dm.n_sink, sl, hps);
  } else if (csize == 1) {
    auto kern = ept == 2 ? select_kernel<2, false> : ept == 8 ? select_kernel<8, false>
                         : ept == 16 ? select_kernel<16, false> : select_kernel<32, false>;
    kern<<<grid, kSelThreads, 0, st>>>(scores, budgets, offsets, kept_idx, rows_cap, n, dm.w, 0, hr.h0, dm.n_sink, sl,
                                       hps);
  } else {
    auto kern = select_kernel<32, true>;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid * csize);
    cfg.blockDim = dim3(kSelThreads);
    cfg.stream = st;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = csize;
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, scores, budgets, offsets, kept_idx, (long long)rows_cap, n,
                                             dm.w, 0, hr.h0, dm.n_sink, sl, hps);
    if (e != cudaSuccess) return e;
  }
  lc.mark("select");
  return cudaGetLastError();
}

cudaError_t launch_gather(const Dims& dm, const int32_t* offsets, const int32_t* kept_idx, const void* k,
                          const void* v, void* k_out, void* v_out, int64_t rows_cap, HeadRange hr, LaunchCtx& lc) {
  cudaStream_t st = lc.st;
  if (rows_cap <= 0) return cudaSuccess;
  const int lpr = (int)(dm.d * dm.esize() / 16);
  switch (lpr) {
    case 8: launch_gather_t<8>(dm, offsets, kept_idx, k, v, k_out, v_out, rows_cap, hr, st); break;
    case 16: launch_gather_t<16>(dm, offsets, kept_idx, k, v, k_out, v_out, rows_cap, hr, st); break;
    default: launch_gather_t<32>(dm, offsets, kept_idx, k, v, k_out, v_out, rows_cap, hr, st); break;
  }
  lc.mark("gather");
  return cudaGetLastError();
}

}  // namespace lukv
