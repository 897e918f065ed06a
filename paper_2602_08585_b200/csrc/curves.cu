// Utility-versus-budget curves of a proxy metric (paper Sec. 3.2: M^pi(k) = the first k positions in the
// ranking of pi; Eq. "head_loss_def": the loss of a retained set is the oracle importance outside it).
// The curve point U(k) is the importance mass of the k highest-ranked positions.  One CTA per head:
//   rank    the order is: sinks first, score descending, lower position first among equals.  Up to 16384
//           positions (the calibration contexts this serves have a few thousand): a bitonic sort in shared
//           memory of 64-bit keys (order-preserving image of the score, then the inverted position), and the
//           importance of the r-th key's position goes to slot r.  Longer heads: every position's rank by
//           counting the positions ahead of it (O(n^2) compares on keys held in shared memory), and the
//           importance of position j goes to slot rank(j).  Ranks are unique either way, so both fill the
//           same array;
//   sum     one thread per curve segment adds its slots in fp64, in order; the running sum over the
//           segments, also in order, gives the curve points, each rounded once to fp32.
#include "common.cuh"

namespace lukv {
namespace {

constexpr int kCurveThreads = 1024;
constexpr int kCurvePer = 4;  // positions ranked together by a thread (one key load serves all of them)

__device__ __forceinline__ uint32_t curve_key(float x, int j, int n_sink) {
  if (j < n_sink) return 0xFFFFFFFFu;
  const uint32_t b = __float_as_uint(x);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);  // order-preserving map float -> uint32
}

// Curve points from the importance in ranking order: one thread per curve segment adds its slots in fp64, in
// order; warp 0 then runs the sum over the segments.  Call with the whole CTA, after a barrier behind the writes of
// `sorted`.
__device__ __forceinline__ void curve_tail(const float* sorted, double* segsum, float* out, int n, int P, int seg,
                                           int tid, int nthreads) {
  const int nseg = P - 1;
  for (int k = tid; k < nseg; k += nthreads) {
    const long long lo = (long long)k * seg, hi = lo + seg;
    const int a = (int)(lo < n ? lo : n), b = (int)(hi < n ? hi : n);
    double acc = 0.0;
    for (int i = a; i < b; ++i) acc = __dadd_rn(acc, (double)sorted[i]);
    segsum[k] = acc;
  }
  __syncthreads();
  // running sum over the segments: warp 0, 32 consecutive segments per step
  if (tid < 32) {
    if (tid == 0) out[0] = 0.f;
    double carry = 0.0;
    for (int k0 = 0; k0 < nseg; k0 += 32) {
      const int k = k0 + tid;
      double v = k < nseg ? segsum[k] : 0.0;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const double o = __shfl_up_sync(0xffffffffu, v, off);
        if (tid >= off) v = __dadd_rn(v, o);
      }
      v = __dadd_rn(v, carry);
      if (k < nseg) out[k + 1] = __double2float_rn(v);
      carry = __shfl_sync(0xffffffffu, v, 31);
    }
  }
}

__global__ void __launch_bounds__(kCurveThreads) build_curves_kernel(const float* __restrict__ scores,
                                                                     const float* __restrict__ importance,
                                                                     float* __restrict__ curves, int n, int P,
                                                                     int seg, int n_sink) {
  extern __shared__ __align__(16) unsigned char curve_smem[];
  const int npad = (n + 3) & ~3;
  uint32_t* keys = reinterpret_cast<uint32_t*>(curve_smem);             // [npad], padding = 0 (ranks last)
  float* sorted = reinterpret_cast<float*>(curve_smem) + npad;          // [npad] importance in ranking order
  double* segsum = reinterpret_cast<double*>(sorted + npad + (npad & 1));  // [P-1], 8-byte aligned
  const int u = blockIdx.x, tid = threadIdx.x;
  const float* sc = scores + (size_t)u * n;
  const float* im = importance + (size_t)u * n;
  for (int j = tid; j < npad; j += kCurveThreads) keys[j] = j < n ? curve_key(sc[j], j, n_sink) : 0u;
  __syncthreads();

  for (int j0 = tid * kCurvePer; j0 < n; j0 += kCurveThreads * kCurvePer) {
    uint32_t mine[kCurvePer];
    int rank[kCurvePer];
#pragma unroll
    for (int i = 0; i < kCurvePer; ++i) {
      mine[i] = j0 + i < n ? keys[j0 + i] : 0u;
      rank[i] = 0;
    }
    // positions ahead of j: a larger key, or an equal key at a lower position
    for (int c = 0; c < npad; c += 4) {
      const uint4 k4 = *reinterpret_cast<const uint4*>(keys + c);
      const uint32_t kk[4] = {k4.x, k4.y, k4.z, k4.w};
#pragma unroll
      for (int i = 0; i < kCurvePer; ++i)
#pragma unroll
        for (int t = 0; t < 4; ++t)
          rank[i] += (kk[t] > mine[i]) || (kk[t] == mine[i] && c + t < j0 + i);
    }
#pragma unroll
    for (int i = 0; i < kCurvePer; ++i)
      if (j0 + i < n) sorted[rank[i]] = im[j0 + i];
  }
  __syncthreads();

  curve_tail(sorted, segsum, curves + (size_t)u * P, n, P, seg, tid, kCurveThreads);
}

constexpr int kSortThreads = 512;
constexpr int kSortMaxN = 16384;  // positions (rounded up to a power of two) the sorting kernel takes

// Sorting variant: comp[r] = (key << 32) | (0xFFFFFFFF - position), sorted descending, so equal keys come out in
// ascending position; padding entries are 0 and end up last.
__global__ void __launch_bounds__(kSortThreads) build_curves_sort_kernel(const float* __restrict__ scores,
                                                                         const float* __restrict__ importance,
                                                                         float* __restrict__ curves, int n, int npow2,
                                                                         int P, int seg, int n_sink) {
  extern __shared__ __align__(16) unsigned char curve_smem[];
  unsigned long long* comp = reinterpret_cast<unsigned long long*>(curve_smem);  // [npow2]
  float* sorted = reinterpret_cast<float*>(comp + npow2);                         // [n + (n & 1)]
  double* segsum = reinterpret_cast<double*>(sorted + n + (n & 1));               // [P-1], 8-byte aligned
  const int u = blockIdx.x, tid = threadIdx.x;
  const float* sc = scores + (size_t)u * n;
  const float* im = importance + (size_t)u * n;
  for (int j = tid; j < npow2; j += kSortThreads)
    comp[j] = j < n ? ((unsigned long long)curve_key(sc[j], j, n_sink) << 32) | (unsigned long long)(0xFFFFFFFFu - (uint32_t)j)
                    : 0ull;
  __syncthreads();
  const int pairs = npow2 >> 1;
  for (int k = 2; k <= npow2; k <<= 1) {
    for (int j = k >> 1, lj = 31 - __clz(j); j > 0; j >>= 1, --lj) {
      for (int t = tid; t < pairs; t += kSortThreads) {
        const int a = ((t >> lj) << (lj + 1)) + (t & (j - 1)), b = a + j;
        const unsigned long long x = comp[a], y = comp[b];
        const bool descending = (a & k) == 0;
        if ((x < y) == descending) {
          comp[a] = y;
          comp[b] = x;
        }
      }
      __syncthreads();
    }
  }
  for (int r = tid; r < n; r += kSortThreads) sorted[r] = im[0xFFFFFFFFu - (uint32_t)comp[r]];
  __syncthreads();
  curve_tail(sorted, segsum, curves + (size_t)u * P, n, P, seg, tid, kSortThreads);
}

int curve_pow2(int n) {
  int p = 2;
  while (p < n) p <<= 1;
  return p;
}
size_t curves_sort_smem_bytes(int n, int P) {
  return (size_t)curve_pow2(n) * 8 + ((size_t)n + (n & 1)) * 4 + (size_t)(P - 1) * 8;
}

}  // namespace

size_t curves_smem_bytes(int n, int P) {
  if (curve_pow2(n) <= kSortMaxN) return curves_sort_smem_bytes(n, P);
  const size_t npad = ((size_t)n + 3) & ~(size_t)3;
  return (2 * npad + (npad & 1)) * 4 + (size_t)(P - 1) * 8;
}

cudaError_t launch_build_curves(const Dims& dm, const float* scores, const float* importance, float* curves,
                                LaunchCtx& lc) {
  const size_t smem = curves_smem_bytes(dm.n, dm.P);
  cudaError_t e;
  if (curve_pow2(dm.n) <= kSortMaxN) {
    if ((e = cudaFuncSetAttribute(build_curves_sort_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) !=
        cudaSuccess)
      return e;
    build_curves_sort_kernel<<<(unsigned)dm.heads(), kSortThreads, smem, lc.st>>>(scores, importance, curves, dm.n,
                                                                                  curve_pow2(dm.n), dm.P, dm.seg,
                                                                                  dm.n_sink);
    lc.mark("build_curves_sort");
    return cudaGetLastError();
  }
  if ((e = cudaFuncSetAttribute(build_curves_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess)
    return e;
  build_curves_kernel<<<(unsigned)dm.heads(), kCurveThreads, smem, lc.st>>>(scores, importance, curves, dm.n, dm.P,
                                                                            dm.seg, dm.n_sink);
  lc.mark("build_curves");
  return cudaGetLastError();
}

}  // namespace lukv
