// KeyDiff proxy scores (the second metric the paper evaluates, pi_2 of Sec. 5.1; recent window 1 in App. E).  The
// paper only names the metric; the formula is the one of the method's own publication:
//   u_j = k_j / max(||k_j||, eps),  a = mean of u_j over all T cached keys of the head,
//   score_j = - <k_j, a> / (max(||k_j||, eps) * max(||a||, eps)),  eps = 1e-8, for the n = T-w rankable positions.
// A key-only scan with no contraction: bound by HBM.  The anchor needs every key of the head before any score, so
// K is read twice; heads are processed in groups whose keys fit L2, so that the second read does not come from HBM.
#include <cooperative_groups.h>

#include <cstdlib>

#include "common.cuh"

namespace lukv {
namespace {

namespace cg = cooperative_groups;

constexpr int kKdThreads = 512;
constexpr int kKdMaxGrid = 2048;  // CTAs of the persistent grid (two per SM)
constexpr float kKdEps = 1e-8f;

template <typename TIn>
struct Vec16;
template <>
struct Vec16<__nv_bfloat16> {
  static constexpr int kElems = 8;
  __device__ static void load(const __nv_bfloat16* p, float (&x)[8]) {
    const uint4 raw = __ldg(reinterpret_cast<const uint4*>(p));
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
  __device__ static void load(const float* p, float (&x)[4]) {
    const float4 raw = __ldg(reinterpret_cast<const float4*>(p));
    x[0] = raw.x, x[1] = raw.y, x[2] = raw.z, x[3] = raw.w;
  }
};

// One persistent cooperative kernel: the grid walks the heads in groups whose keys fit L2.  The rows of a group
// (heads x T, one after the other) are cut into equal slices, one per CTA, so that every SM streams the same share
// whatever T is.  For a group a CTA first sums the unit keys of its slice -- one partial sum per head the slice
// touches ("piece") --, the grid meets at a barrier, and the CTA scores the same slice, first adding the pieces
// of the head in order (the anchor).  Piece ids: CTA b's piece of the group's u-th head is b + u, which is unique
// and ascending along the rows; the pieces of two consecutive groups live in two halves of the scratch, so that a
// CTA already summing the next group does not overwrite what a slower one still reads.
// LPR lanes share one key row, 16 bytes each; a warp takes 32/LPR rows at a time and keeps four loads in flight.
template <typename TIn, int LPR>
__global__ void __launch_bounds__(kKdThreads, 2) keydiff_kernel(const TIn* __restrict__ k, float* partial,
                                                                float* __restrict__ scores, int T, int n, int heads,
                                                                int group, int half_pieces) {
  constexpr int E = Vec16<TIn>::kElems, D = LPR * E, kRowsPerIter = 32 / LPR, kWarps = kKdThreads / 32, kUnroll = 4;
  constexpr int kTrip = kUnroll * kWarps * kRowsPerIter;
  constexpr int kSplit = kKdThreads / D;  // threads per column when the pieces of a head are added
  static_assert(kSplit >= 1 && kSplit <= kWarps, "the split sums reuse red");
  __shared__ float red[kWarps][D];
  __shared__ float anchor_s[D];
  __shared__ float inv_an_s;
  cg::grid_group grid = cg::this_grid();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, sub = lane / LPR, part = lane % LPR;
  int parity = 0;
  for (int h0 = 0; h0 < heads; h0 += group, parity ^= 1) {
    const int nh = min(group, heads - h0);
    const long long rows = (long long)nh * T;
    long long per = (rows + gridDim.x - 1) / gridDim.x;
    per = (per + kWarps * kRowsPerIter - 1) / (kWarps * kRowsPerIter) * (kWarps * kRowsPerIter);
    const long long lo = min(rows, (long long)blockIdx.x * per), hi = min(rows, lo + per);
    float* pieces = partial + (size_t)parity * half_pieces * D;
    // ---- sums of unit keys, one piece per head of the slice
    for (long long at = lo; at < hi;) {
      const int ul = (int)(at / T);
      const int j_begin = (int)(at - (long long)ul * T), j_end = (int)min((long long)T, hi - (long long)ul * T);
      const TIn* base = k + (size_t)(h0 + ul) * T * D;
      float acc[E];
#pragma unroll
      for (int e = 0; e < E; ++e) acc[e] = 0.f;
      for (int j0 = j_begin + warp * kRowsPerIter; j0 < j_end; j0 += kTrip) {
        float x[kUnroll][E];
#pragma unroll
        for (int r = 0; r < kUnroll; ++r) {
          const int j = j0 + r * kWarps * kRowsPerIter + sub;
#pragma unroll
          for (int e = 0; e < E; ++e) x[r][e] = 0.f;
          if (j < j_end) Vec16<TIn>::load(base + (size_t)j * D + part * E, x[r]);
        }
#pragma unroll
        for (int r = 0; r < kUnroll; ++r) {
          float ss = 0.f;
#pragma unroll
          for (int e = 0; e < E; ++e) ss = fmaf(x[r][e], x[r][e], ss);
#pragma unroll
          for (int off = 1; off < LPR; off <<= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
          const float inv = 1.f / fmaxf(sqrtf(ss), kKdEps);  // rows past the piece are all zero and add nothing
#pragma unroll
          for (int e = 0; e < E; ++e) acc[e] = fmaf(x[r][e], inv, acc[e]);
        }
      }
      // the rows a warp holds side by side, then the warps, in a fixed order
#pragma unroll
      for (int off = LPR; off < 32; off <<= 1)
#pragma unroll
        for (int e = 0; e < E; ++e) acc[e] += __shfl_xor_sync(0xffffffffu, acc[e], off);
      __syncthreads();  // red is free again
      if (sub == 0)
#pragma unroll
        for (int e = 0; e < E; ++e) red[warp][part * E + e] = acc[e];
      __syncthreads();
      for (int c = threadIdx.x; c < D; c += kKdThreads) {
        float s = 0.f;
#pragma unroll
        for (int wv = 0; wv < kWarps; ++wv) s += red[wv][c];
        __stcg(pieces + (size_t)(blockIdx.x + ul) * D + c, s);
      }
      at = (long long)ul * T + j_end;
    }
    __threadfence();
    grid.sync();
    // ---- scores of the same slice
    for (long long at = lo; at < hi;) {
      const int ul = (int)(at / T);
      const int j_begin = (int)(at - (long long)ul * T), j_end = (int)min((long long)T, hi - (long long)ul * T);
      at = (long long)ul * T + j_end;
      if (j_begin >= n) continue;  // only window rows of this head in the slice
      // anchor = mean of the unit keys = the head's pieces added in order / T, and its norm
      const int first = (int)(((long long)ul * T) / per), last = (int)((((long long)ul + 1) * T - 1) / per);
      // kSplit threads share a column: thread g of them adds pieces first+g, first+g+kSplit, ...; then in order
      __syncthreads();
      {
        const int c = threadIdx.x % D, g = threadIdx.x / D;
        float s = 0.f;
#pragma unroll 4
        for (int b = first + g; b <= last; b += kSplit) s += __ldcg(pieces + (size_t)(b + ul) * D + c);
        red[g][c] = s;
      }
      __syncthreads();
      if (threadIdx.x < D) {
        float s = 0.f;
#pragma unroll
        for (int g = 0; g < kSplit; ++g) s += red[g][threadIdx.x];
        anchor_s[threadIdx.x] = s / (float)T;
      }
      __syncthreads();
      if (threadIdx.x < 32) {
        float n2 = 0.f;
        for (int i = lane; i < D; i += 32) n2 = fmaf(anchor_s[i], anchor_s[i], n2);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) n2 += __shfl_xor_sync(0xffffffffu, n2, off);
        if (lane == 0) inv_an_s = 1.f / fmaxf(sqrtf(n2), kKdEps);
      }
      __syncthreads();
      float av[E];
#pragma unroll
      for (int e = 0; e < E; ++e) av[e] = anchor_s[part * E + e];
      const float inv_an = inv_an_s;
      const int jn_end = min(j_end, n);
      const TIn* base = k + (size_t)(h0 + ul) * T * D;
      float* out = scores + (size_t)(h0 + ul) * n;
      for (int j0 = j_begin + warp * kRowsPerIter; j0 < jn_end; j0 += kTrip) {
        float x[kUnroll][E];
#pragma unroll
        for (int r = 0; r < kUnroll; ++r) {
          const int j = j0 + r * kWarps * kRowsPerIter + sub;
#pragma unroll
          for (int e = 0; e < E; ++e) x[r][e] = 0.f;
          if (j < jn_end) Vec16<TIn>::load(base + (size_t)j * D + part * E, x[r]);
        }
#pragma unroll
        for (int r = 0; r < kUnroll; ++r) {
          const int j = j0 + r * kWarps * kRowsPerIter + sub;
          float ss = 0.f, dot = 0.f;
#pragma unroll
          for (int e = 0; e < E; ++e) {
            ss = fmaf(x[r][e], x[r][e], ss);
            dot = fmaf(x[r][e], av[e], dot);
          }
#pragma unroll
          for (int off = 1; off < LPR; off <<= 1) {
            ss += __shfl_xor_sync(0xffffffffu, ss, off);
            dot += __shfl_xor_sync(0xffffffffu, dot, off);
          }
          if (part == 0 && j < jn_end) out[j] = -dot * inv_an / fmaxf(sqrtf(ss), kKdEps);
        }
      }
    }
  }
}

// heads per group: their keys stay in L2 between the two reads (LUKV_KEYDIFF_GROUP_MB overrides the size for
// tuning runs)
int keydiff_group(const Dims& dm, size_t elem) {
  const char* env = getenv("LUKV_KEYDIFF_GROUP_MB");
  const int env_mb = env ? atoi(env) : 0;
  const size_t group_bytes = (size_t)(env_mb >= 1 && env_mb <= 4096 ? env_mb : 4096) << 20;
  const size_t g = group_bytes / ((size_t)dm.T * dm.d * elem);
  const size_t cap = (size_t)dm.heads() < (size_t)kKdMaxGrid ? (size_t)dm.heads() : (size_t)kKdMaxGrid;
  return (int)(g < 1 ? 1 : g > cap ? cap : g);
}

template <typename TIn, int LPR>
cudaError_t launch_keydiff_t(const Dims& dm, const void* k, float* scores, float* partial, LaunchCtx& lc) {
  auto kern = keydiff_kernel<TIn, LPR>;
  int dev = 0, sms = 0, per_sm = 0;
  cudaError_t e;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
  if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kKdThreads, 0)) != cudaSuccess) return e;
  if (per_sm < 1) return cudaErrorLaunchOutOfResources;
  int group = keydiff_group(dm, sizeof(TIn));
  const int heads = (int)dm.heads();
  // a slice is at least one trip of the CTA: tiny problems get a smaller grid
  const long long slices = ((long long)group * dm.T + kKdThreads / LPR - 1) / (kKdThreads / LPR);
  long long grid = (long long)sms * per_sm;
  grid = grid > kKdMaxGrid ? kKdMaxGrid : grid;
  grid = grid > slices ? slices : grid;
  const TIn* kp = (const TIn*)k;
  int T = dm.T, n = dm.n, half = kKdMaxGrid + group;
  void* params[] = {(void*)&kp,    (void*)&partial, (void*)&scores, (void*)&T,
                    (void*)&n,     (void*)&heads,   (void*)&group,  (void*)&half};
  // cooperative launch: the grid meets at a barrier between the two reads of a group
  e = cudaLaunchCooperativeKernel((const void*)kern, dim3((unsigned)grid), dim3(kKdThreads), params, 0, lc.st);
  lc.mark("keydiff");
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace

// fp32 scratch of the KeyDiff scorer: the pieces of two consecutive groups, [2][grid + heads of a group][d], at
// the largest grid and group
size_t keydiff_scratch_bytes(const Dims& dm) {
  const size_t group = (size_t)dm.heads() < (size_t)kKdMaxGrid ? (size_t)dm.heads() : (size_t)kKdMaxGrid;
  return (size_t)2 * (kKdMaxGrid + group) * dm.d * sizeof(float);
}

cudaError_t launch_keydiff(const Dims& dm, const void* k, float* scores, float* scratch, LaunchCtx& lc) {
  if (dm.dtype == LUKV_DTYPE_BF16)
    return dm.d == 128 ? launch_keydiff_t<__nv_bfloat16, 16>(dm, k, scores, scratch, lc)
                       : launch_keydiff_t<__nv_bfloat16, 8>(dm, k, scores, scratch, lc);
  return dm.d == 128 ? launch_keydiff_t<float, 32>(dm, k, scores, scratch, lc)
                     : launch_keydiff_t<float, 16>(dm, k, scores, scratch, lc);
}

}  // namespace lukv
