// Utility-versus-budget curves of a proxy metric (paper Sec. 3.2: M^pi(k) = the first k positions in the
// ranking of pi; Eq. "head_loss_def": the loss of a retained set is the oracle importance outside it).
// The curve point U(k) is the importance mass of the k highest-ranked positions.  One CTA per head:
//   rank    every position's place in the order (sinks first, score descending, lower position first
//           among equals) by counting the positions ahead of it -- O(n^2) compares on keys held in
//           shared memory, which for the calibration contexts this serves (a few thousand tokens)
//           beats a sort's passes and needs no scratch memory;
//   scatter the importance of position j goes to slot rank(j) of a shared array (ranks are unique);
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

  const int nseg = P - 1;
  for (int k = tid; k < nseg; k += kCurveThreads) {
    const long long lo = (long long)k * seg, hi = lo + seg;
    const int a = (int)(lo < n ? lo : n), b = (int)(hi < n ? hi : n);
    double acc = 0.0;
    for (int i = a; i < b; ++i) acc = __dadd_rn(acc, (double)sorted[i]);
    segsum[k] = acc;
  }
  __syncthreads();
  // running sum over the segments: warp 0, 32 consecutive segments per step
  if (tid < 32) {
    float* out = curves + (size_t)u * P;
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

}  // namespace

size_t curves_smem_bytes(int n, int P) {
  const size_t npad = ((size_t)n + 3) & ~(size_t)3;
  return (2 * npad + (npad & 1)) * 4 + (size_t)(P - 1) * 8;
}

cudaError_t launch_build_curves(const Dims& dm, const float* scores, const float* importance, float* curves,
                                LaunchCtx& lc) {
  const size_t smem = curves_smem_bytes(dm.n, dm.P);
  cudaError_t e;
  if ((e = cudaFuncSetAttribute(build_curves_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess)
    return e;
  build_curves_kernel<<<(unsigned)dm.heads(), kCurveThreads, smem, lc.st>>>(scores, importance, curves, dm.n, dm.P,
                                                                            dm.seg, dm.n_sink);
  lc.mark("build_curves");
  return cudaGetLastError();
}

}  // namespace lukv
