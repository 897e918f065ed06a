// KeyDiff proxy scores (the second metric the paper evaluates, pi_2 of Sec. 5.1; recent window 1 in App. E).  The
// paper only names the metric; the formula is the one of the method's own publication:
//   u_j = k_j / max(||k_j||, eps),  a = mean of u_j over all T cached keys of the head,
//   score_j = - <k_j, a> / (max(||k_j||, eps) * max(||a||, eps)),  eps = 1e-8, for the n = T-w rankable positions.
// A key-only scan with no contraction: bound by HBM.  The anchor needs every key of the head before any score, so
// K is read twice.  The kernel can walk the heads in groups, the CTAs alternating between the first read of one
// group and the second read of the group before it (which L2 then serves); by default there is one group.
#include <cstdlib>

#include "tc_ptx.cuh"

namespace lukv {
namespace {

constexpr int kKdConsumerWarps = 8;
constexpr int kKdConsumers = kKdConsumerWarps * 32;
constexpr int kKdThreads = kKdConsumers + 32;  // + the warp whose first lane issues the bulk copies
constexpr int kKdStageRows = 64;               // key rows per shared-memory stage: 8 per consumer warp
constexpr int kKdRingBytes = 96 * 1024;        // ring of stages per CTA; two CTAs per SM
constexpr int kKdMaxGrid = 2048;               // CTAs of the persistent grid
constexpr int kKdLanesPerRow = 4;
constexpr float kKdEps = 1e-8f;
constexpr int kKdBarConsumers = 1;             // named barrier of the consumer warps

template <typename TIn>
struct Vec16;
template <>
struct Vec16<__nv_bfloat16> {
  static constexpr int kElems = 8;
  __device__ static void load(const unsigned char* p, float (&x)[8]) {
    const uint4 raw = *reinterpret_cast<const uint4*>(p);
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 f = __bfloat1622float2(h[i]);
      x[2 * i] = f.x;
      x[2 * i + 1] = f.y;
    }
  }
};
template <>
struct Vec16<float> {
  static constexpr int kElems = 4;
  __device__ static void load(const unsigned char* p, float (&x)[4]) {
    const float4 raw = *reinterpret_cast<const float4*>(p);
    x[0] = raw.x, x[1] = raw.y, x[2] = raw.z, x[3] = raw.w;
  }
};

struct KdArgs {
  const unsigned char* k;  // [heads][T][d]
  float* scores;           // [heads][n]
  float* pieces;           // [2][kKdMaxGrid + group][d]: partial sums of unit keys, by parity of the group
  float* anchors;          // [heads][d]   mean unit key
  float* inv_norm;         // [heads]      1 / max(||anchor||, eps)
  int* head_count;         // [heads]      pieces delivered; one more once the anchor is published.  Starts at 0.
  int32_t* dev_status;     // may be null
  int T, n, heads, group;
  uint32_t spin_limit;
  int drop_head;           // test hook: this head's anchor is never published (-1: none)
};

__device__ __forceinline__ int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// The slice of a group's rows (heads x T, one head after the other) that a CTA owns: equal slices, whole stages.
struct KdSlice {
  int h0, nh;
  long long per, lo, hi;
};
__device__ __forceinline__ KdSlice kd_slice(const KdArgs& a, int g) {
  KdSlice s;
  s.h0 = g * a.group;
  s.nh = min(a.group, a.heads - s.h0);
  const long long rows = (long long)s.nh * a.T;
  s.per = (rows + gridDim.x - 1) / gridDim.x;
  s.per = (s.per + kKdStageRows - 1) / kKdStageRows * kKdStageRows;
  s.lo = min(rows, (long long)blockIdx.x * s.per);
  s.hi = min(rows, s.lo + s.per);
  return s;
}

// A lane's share of one key row out of a stage: V loads of 16 bytes (zeros for a row the stage does not hold).
// Lane l of the four that share the row reads the 16-byte parts 4i + l; odd rows take i in rotated order so that
// the two rows of a quarter-warp fall into different banks.
template <typename TIn, int V>
__device__ __forceinline__ void kd_load_row(const unsigned char* row, bool present, int l, int odd_row,
                                            float (&x)[V][Vec16<TIn>::kElems]) {
#pragma unroll
  for (int i = 0; i < V; ++i) {
#pragma unroll
    for (int e = 0; e < Vec16<TIn>::kElems; ++e) x[i][e] = 0.f;
    if (present) Vec16<TIn>::load(row + (4 * ((i + odd_row) % V) + l) * 16, x[i]);
  }
}

// One persistent cooperative kernel (cooperative only so that all CTAs are resident: they wait for one another's
// partial sums).  A CTA owns the same slice of every group.  Its "sum" step of a group adds the unit keys of the
// slice, one partial sum ("piece") per head the slice touches; the CTA that delivers the last piece of a head adds
// the pieces in order and publishes the anchor.  Its "score" step of a group re-reads the slice (from L2) and
// scores it against the published anchors.  Even CTAs run sum(g), score(g-1), sum(g+1), ...; odd CTAs score first,
// so that at any time half of the grid reads HBM and half reads L2.  Piece ids: CTA b's piece of the u-th head of
// a group is b + u, unique and ascending along the rows.  A piece slot is written again two groups later, after
// its CTA has waited, in the score step in between, for the anchors made from it.
// Rows arrive in a ring of shared-memory stages filled by bulk copies that one producer lane issues as far ahead
// as the ring allows, across the two kinds of step.
template <typename TIn, int D>
__global__ void __launch_bounds__(kKdThreads, 2) keydiff_kernel(const KdArgs a) {
  constexpr int E = Vec16<TIn>::kElems;
  constexpr int kRowBytes = D * (int)sizeof(TIn);
  constexpr int kStageBytes = kKdStageRows * kRowBytes;
  constexpr int kStages = kKdRingBytes / kStageBytes;
  constexpr int V = kRowBytes / (16 * kKdLanesPerRow);  // 16-byte loads per lane and row
  constexpr int kSplit = kKdConsumers / D;              // threads per column when the pieces of a head are added
  static_assert(V >= 2 && V % 2 == 0 && kStages >= 2 && kSplit >= 1 && kSplit <= 2 * kKdConsumerWarps, "shape");
  extern __shared__ __align__(128) unsigned char ring[];
  __shared__ __align__(8) uint64_t bars[2 * kStages];  // full[kStages], empty[kStages]
  __shared__ float red[2 * kKdConsumerWarps][D];
  __shared__ float anchor_s[D];
  __shared__ int last_s;
  __shared__ int abort_s;
  volatile int* abort_flag = &abort_s;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = (a.heads + a.group - 1) / a.group;
  const bool odd_cta = blockIdx.x & 1;
  if (threadIdx.x == 0) {
    abort_s = 0;
    for (int s = 0; s < kStages; ++s) {
      mbar_init(smem_u32(&bars[s]), 1);
      mbar_init(smem_u32(&bars[kStages + s]), kKdConsumerWarps);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  if (warp == kKdConsumerWarps) {
    // ---- producer: the same walk over steps, pieces and stages as the consumers
    if (lane != 0) return;
    uint32_t cnt = 0;
    bool ok = true;
    for (int it = 0; it <= G && ok; ++it) {
      for (int half = 0; half < 2 && ok; ++half) {
        const bool sum_step = (half == 0) != odd_cta;
        const int g = sum_step ? it : it - 1;
        if (g < 0 || g >= G) continue;
        const KdSlice sl = kd_slice(a, g);
        for (long long at = sl.lo; at < sl.hi && ok;) {
          const int ul = (int)(at / a.T);
          const int j_begin = (int)(at - (long long)ul * a.T);
          const int j_end_all = (int)min((long long)a.T, sl.hi - (long long)ul * a.T);
          const int j_end = sum_step ? j_end_all : min(j_end_all, a.n);
          const unsigned char* base = a.k + (size_t)(sl.h0 + ul) * a.T * kRowBytes;
          for (int j = j_begin; j < j_end; j += kKdStageRows, ++cnt) {
            const uint32_t s = cnt % kStages, use = cnt / kStages;
            ok = mbar_wait(smem_u32(&bars[kStages + s]), (use & 1) ^ 1, abort_flag, a.dev_status, a.spin_limit);
            if (!ok) break;
            const uint32_t bytes = (uint32_t)min(kKdStageRows, j_end - j) * kRowBytes;
            mbar_expect_tx(smem_u32(&bars[s]), bytes);
            bulk_load(smem_u32(ring + (size_t)s * kStageBytes), base + (size_t)j * kRowBytes, bytes,
                      smem_u32(&bars[s]));
          }
          at = (long long)ul * a.T + j_end_all;
        }
      }
    }
    if (!ok) {
      // giving up: no copy of this CTA may still be in flight when it exits
      for (uint32_t back = 1; back <= (uint32_t)kStages && back <= cnt; ++back) {
        const uint32_t c = cnt - back, s = c % kStages, use = c / kStages;
        for (uint32_t i = 0; i < a.spin_limit && !mbar_try_wait(smem_u32(&bars[s]), use & 1); ++i) __nanosleep(64);
      }
    }
    return;
  }

  // ---- consumers.  Nothing below leaves a loop early: once the abort flag is up every wait returns at once, the
  // named barriers stay matched, and the walk ends after arithmetic on whatever the stages hold.
  const int l = lane & (kKdLanesPerRow - 1), r = lane >> 2, odd_row = r & 1;
  const int row_in_stage = warp * 8 + r;
  uint32_t cnt = 0;
  for (int it = 0; it <= G; ++it) {
    for (int half = 0; half < 2; ++half) {
      const bool sum_step = (half == 0) != odd_cta;
      const int g = sum_step ? it : it - 1;
      if (g < 0 || g >= G) continue;
      const KdSlice sl = kd_slice(a, g);
      float* pieces = a.pieces + (size_t)(g & 1) * (kKdMaxGrid + a.group) * D;
      for (long long at = sl.lo; at < sl.hi;) {
        const int ul = (int)(at / a.T), u = sl.h0 + ul;
        const int j_begin = (int)(at - (long long)ul * a.T);
        const int j_end_all = (int)min((long long)a.T, sl.hi - (long long)ul * a.T);
        at = (long long)ul * a.T + j_end_all;
        // CTAs that hold a piece of this head
        const int first = (int)(((long long)ul * a.T) / sl.per);
        const int last = (int)((((long long)ul + 1) * a.T - 1) / sl.per);
        if (sum_step) {
          float acc[V][E];
#pragma unroll
          for (int i = 0; i < V; ++i)
#pragma unroll
            for (int e = 0; e < E; ++e) acc[i][e] = 0.f;
          for (int j = j_begin; j < j_end_all; j += kKdStageRows, ++cnt) {
            const uint32_t s = cnt % kStages, use = cnt / kStages;
            mbar_wait(smem_u32(&bars[s]), use & 1, abort_flag, a.dev_status, a.spin_limit);
            float x[V][E];
            kd_load_row<TIn, V>(ring + (size_t)s * kStageBytes + (size_t)row_in_stage * kRowBytes,
                                j + row_in_stage < j_end_all, l, odd_row, x);
            float ssv[V];
#pragma unroll
            for (int i = 0; i < V; ++i) {
              ssv[i] = 0.f;
#pragma unroll
              for (int e = 0; e < E; ++e) ssv[i] = fmaf(x[i][e], x[i][e], ssv[i]);
            }
            float ss = 0.f;
#pragma unroll
            for (int i = 0; i < V; ++i) ss += ssv[i];
            ss += __shfl_xor_sync(0xffffffffu, ss, 1);
            ss += __shfl_xor_sync(0xffffffffu, ss, 2);
            const float inv = 1.f / fmaxf(sqrtf(ss), kKdEps);  // an absent row is all zero and adds nothing
#pragma unroll
            for (int i = 0; i < V; ++i)
#pragma unroll
              for (int e = 0; e < E; ++e) acc[i][e] = fmaf(x[i][e], inv, acc[i][e]);
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&bars[kStages + s]), 1);
          }
          // rows of equal parity a warp holds side by side, then warps and parities in a fixed order
#pragma unroll
          for (int i = 0; i < V; ++i)
#pragma unroll
            for (int e = 0; e < E; ++e) {
              acc[i][e] += __shfl_xor_sync(0xffffffffu, acc[i][e], 8);
              acc[i][e] += __shfl_xor_sync(0xffffffffu, acc[i][e], 16);
            }
          bar_sync(kKdBarConsumers, kKdConsumers);  // red is free again
          if (r < 2)
#pragma unroll
            for (int i = 0; i < V; ++i)
#pragma unroll
              for (int e = 0; e < E; ++e) red[warp * 2 + odd_row][(4 * ((i + odd_row) % V) + l) * E + e] = acc[i][e];
          bar_sync(kKdBarConsumers, kKdConsumers);
          for (int c = threadIdx.x; c < D; c += kKdConsumers) {
            float s = 0.f;
#pragma unroll
            for (int p = 0; p < 2 * kKdConsumerWarps; ++p) s += red[p][c];
            __stcg(pieces + (size_t)(blockIdx.x + ul) * D + c, s);
            __threadfence();
          }
          bar_sync(kKdBarConsumers, kKdConsumers);
          if (threadIdx.x == 0) last_s = atom_add_acq_rel(a.head_count + u, 1) == last - first;
          bar_sync(kKdBarConsumers, kKdConsumers);
          if (last_s) {
            // this CTA delivered the head's last piece: anchor = the pieces added in order / T, and its norm.
            // kSplit threads share a column: thread q of them adds pieces first+q, first+q+kSplit, ...
            {
              const int c = threadIdx.x % D, q = threadIdx.x / D;
              float s = 0.f;
#pragma unroll 8
              for (int b = first + q; b <= last; b += kSplit) s += __ldcg(pieces + (size_t)(b + ul) * D + c);
              red[q][c] = s;
            }
            bar_sync(kKdBarConsumers, kKdConsumers);
            if (threadIdx.x < D) {
              float s = 0.f;
#pragma unroll
              for (int q = 0; q < kSplit; ++q) s += red[q][threadIdx.x];
              s /= (float)a.T;
              anchor_s[threadIdx.x] = s;
              __stcg(a.anchors + (size_t)u * D + threadIdx.x, s);
              __threadfence();
            }
            bar_sync(kKdBarConsumers, kKdConsumers);
            if (threadIdx.x < 32) {
              float n2 = 0.f;
              for (int i = lane; i < D; i += 32) n2 = fmaf(anchor_s[i], anchor_s[i], n2);
#pragma unroll
              for (int off = 16; off > 0; off >>= 1) n2 += __shfl_xor_sync(0xffffffffu, n2, off);
              if (lane == 0) {
                __stcg(a.inv_norm + u, 1.f / fmaxf(sqrtf(n2), kKdEps));
                __threadfence();
                if (u != a.drop_head) atom_add_acq_rel(a.head_count + u, 1);
              }
            }
          }
        } else {
          // wait for the head's anchor (published during the sum step of this group, one step ago)
          if (threadIdx.x == 0) {
            bool have = false;
            for (uint32_t i = 0; i < a.spin_limit && !*abort_flag; ++i) {
              if ((have = ld_acquire(a.head_count + u) == last - first + 2)) break;
              __nanosleep(64);
            }
            if (!have && !*abort_flag) raise_abort(abort_flag, a.dev_status);
          }
          bar_sync(kKdBarConsumers, kKdConsumers);
          float av[V][E];
#pragma unroll
          for (int i = 0; i < V; ++i)
#pragma unroll
            for (int e = 0; e < E; ++e)
              av[i][e] = __ldcg(a.anchors + (size_t)u * D + (4 * ((i + odd_row) % V) + l) * E + e);
          const float inv_an = __ldcg(a.inv_norm + u);
          const int j_end = min(j_end_all, a.n);
          float* out = a.scores + (size_t)u * a.n;
          for (int j = j_begin; j < j_end; j += kKdStageRows, ++cnt) {
            const uint32_t s = cnt % kStages, use = cnt / kStages;
            mbar_wait(smem_u32(&bars[s]), use & 1, abort_flag, a.dev_status, a.spin_limit);
            const bool present = j + row_in_stage < j_end;
            float x[V][E];
            kd_load_row<TIn, V>(ring + (size_t)s * kStageBytes + (size_t)row_in_stage * kRowBytes, present, l,
                                odd_row, x);
            float ssv[V], dotv[V];
#pragma unroll
            for (int i = 0; i < V; ++i) {
              ssv[i] = 0.f, dotv[i] = 0.f;
#pragma unroll
              for (int e = 0; e < E; ++e) {
                ssv[i] = fmaf(x[i][e], x[i][e], ssv[i]);
                dotv[i] = fmaf(x[i][e], av[i][e], dotv[i]);
              }
            }
            float ss = 0.f, dot = 0.f;
#pragma unroll
            for (int i = 0; i < V; ++i) ss += ssv[i], dot += dotv[i];
            ss += __shfl_xor_sync(0xffffffffu, ss, 1);
            dot += __shfl_xor_sync(0xffffffffu, dot, 1);
            ss += __shfl_xor_sync(0xffffffffu, ss, 2);
            dot += __shfl_xor_sync(0xffffffffu, dot, 2);
            if (l == 0 && present) out[j + row_in_stage] = -dot * inv_an / fmaxf(sqrtf(ss), kKdEps);
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&bars[kStages + s]), 1);
          }
        }
      }
    }
  }
}

// Heads per group.  By default a group is as many heads as the piece slots allow, i.e. normally all of them: K is
// then read twice from HBM, at the rate of a plain copy.  Groups small enough for L2 to serve the second read
// (LUKV_KEYDIFF_GROUP_MB sets the group's size in MB of keys) were slower on B200 at every size tried: a step of a
// 40 MB group streams for 6 us, while the hand-over of the partial sums between the CTAs of a head takes longer,
// and L2 cannot hold enough groups in flight to hide it.
int keydiff_group(const Dims& dm) {
  const char* env = getenv("LUKV_KEYDIFF_GROUP_MB");
  const int env_mb = env ? atoi(env) : 0;
  const size_t cap = (size_t)dm.heads() < (size_t)kKdMaxGrid ? (size_t)dm.heads() : (size_t)kKdMaxGrid;
  if (env_mb < 1 || env_mb > 4096) return (int)cap;
  const size_t g = ((size_t)env_mb << 20) / ((size_t)dm.T * dm.d * dm.esize());
  return (int)(g < 1 ? 1 : g > cap ? cap : g);
}

size_t kd_align(size_t x) { return (x + 255) & ~(size_t)255; }
size_t kd_pieces_bytes(const Dims& dm) {
  const size_t group = (size_t)dm.heads() < (size_t)kKdMaxGrid ? (size_t)dm.heads() : (size_t)kKdMaxGrid;
  return kd_align((size_t)2 * (kKdMaxGrid + group) * dm.d * sizeof(float));
}
size_t kd_anchor_bytes(const Dims& dm) { return kd_align((size_t)dm.heads() * dm.d * sizeof(float)); }
size_t kd_head_bytes(const Dims& dm) { return kd_align((size_t)dm.heads() * sizeof(float)); }

template <typename TIn, int D>
cudaError_t launch_keydiff_t(const Dims& dm, const void* k, float* scores, float* scratch, int32_t* dev_status,
                             int spare_sms, LaunchCtx& lc) {
  auto kern = keydiff_kernel<TIn, D>;
  int dev = 0, sms = 0, per_sm = 0;
  cudaError_t e;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kKdRingBytes)) != cudaSuccess)
    return e;
  if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kKdThreads, kKdRingBytes)) != cudaSuccess)
    return e;
  if (per_sm < 1) return cudaErrorLaunchOutOfResources;
  if (spare_sms > 0 && sms > 8 * spare_sms) sms -= spare_sms;  // kernels of another stream keep these
  KdArgs a;
  unsigned char* sc = reinterpret_cast<unsigned char*>(scratch);
  a.k = static_cast<const unsigned char*>(k);
  a.scores = scores;
  a.pieces = reinterpret_cast<float*>(sc);
  a.anchors = reinterpret_cast<float*>(sc + kd_pieces_bytes(dm));
  a.inv_norm = reinterpret_cast<float*>(sc + kd_pieces_bytes(dm) + kd_anchor_bytes(dm));
  a.head_count = reinterpret_cast<int*>(sc + kd_pieces_bytes(dm) + kd_anchor_bytes(dm) + kd_head_bytes(dm));
  a.dev_status = dev_status;
  a.T = dm.T, a.n = dm.n, a.heads = (int)dm.heads(), a.group = keydiff_group(dm);
  score_test_hooks(&a.spin_limit, &a.drop_head);
  if ((e = cudaMemsetAsync(a.head_count, 0, (size_t)a.heads * sizeof(int), lc.st)) != cudaSuccess) return e;
  // a slice is at least one stage: small problems get a smaller grid
  const long long slices = ((long long)a.group * dm.T + kKdStageRows - 1) / kKdStageRows;
  long long grid = (long long)sms * (per_sm > 2 ? 2 : per_sm);
  grid = grid > kKdMaxGrid ? kKdMaxGrid : grid;
  grid = grid > slices ? slices : grid;
  void* params[] = {(void*)&a};
  e = cudaLaunchCooperativeKernel((const void*)kern, dim3((unsigned)grid), dim3(kKdThreads), params, kKdRingBytes,
                                  lc.st);
  lc.mark("keydiff");
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace

// scratch of the KeyDiff scorer: pieces, anchors, their norms, the per-head counters
size_t keydiff_scratch_bytes(const Dims& dm) {
  return kd_pieces_bytes(dm) + kd_anchor_bytes(dm) + 2 * kd_head_bytes(dm);
}

cudaError_t launch_keydiff(const Dims& dm, const void* k, float* scores, float* scratch, int32_t* dev_status,
                           int spare_sms, LaunchCtx& lc) {
  if (dm.dtype == LUKV_DTYPE_BF16)
    return dm.d == 128 ? launch_keydiff_t<__nv_bfloat16, 128>(dm, k, scores, scratch, dev_status, spare_sms, lc)
                       : launch_keydiff_t<__nv_bfloat16, 64>(dm, k, scores, scratch, dev_status, spare_sms, lc);
  return dm.d == 128 ? launch_keydiff_t<float, 128>(dm, k, scores, scratch, dev_status, spare_sms, lc)
                     : launch_keydiff_t<float, 64>(dm, k, scores, scratch, dev_status, spare_sms, lc);
}

}  // namespace lukv
