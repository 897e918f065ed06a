// Exact solution of the allocation problem on the curves as given (paper Sec. 4.2, Eq.
// "combinatorial_optimization"; the paper names the exact solver as the point of comparison for its
// relaxation): the multiple-choice-knapsack recursion over the heads,
//     f_h(x) = max over b in [0, min(x, n)] of  f_{h-1}(x - b) + U_h(b),      f_{-1}(0) = 0,
// at token resolution (curve point b = utility of keeping b tokens).  One launch per head; a thread owns
// four budgets x and walks b upwards, so the smallest b wins a tie; the argmax of every (h, x) is kept for
// the walk back from x = B.  Only the states that can still reach sum b = B are evaluated: after head h,
// x lies in [B - (N-1-h)*n, (h+1)*n].
#include <math.h>

#include "common.cuh"

namespace lukv {
namespace {

constexpr int kDpThreads = 256;
constexpr int kDpPer = 4;                       // budgets per thread
constexpr int kDpTile = kDpThreads * kDpPer;    // budgets per CTA
constexpr int kDpChunk = 1024;                  // values of b staged at a time

__global__ void dp_init_kernel(float* f, long long count) {
  const long long x = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (x < count) f[x] = x == 0 ? 0.f : -INFINITY;
}

// prev holds f_{h-1} on [plo, phi] (anything outside counts as -inf); next receives f_h on [lo, hi].
__global__ void __launch_bounds__(kDpThreads) dp_step_kernel(const float* __restrict__ U, const float* __restrict__ prev,
                                                             float* __restrict__ next,
                                                             unsigned short* __restrict__ choice, int n, long long lo,
                                                             long long hi, long long plo, long long phi) {
  __shared__ float sU[kDpChunk];
  __shared__ float sF[kDpTile + kDpChunk];
  const int tid = threadIdx.x;
  const long long xbase = lo + (long long)blockIdx.x * kDpTile;
  float best[kDpPer];
  int arg[kDpPer];
#pragma unroll
  for (int r = 0; r < kDpPer; ++r) {
    best[r] = -INFINITY;
    arg[r] = 0;
  }
  // b can only matter while x - b stays inside [plo, phi] for some x of this tile
  const long long xlast = min(hi, xbase + kDpTile - 1);
  long long bmin = max(0LL, xbase - phi), bmax = min((long long)n, xlast - plo);
  for (long long b0 = bmin; b0 <= bmax; b0 += kDpChunk) {
    __syncthreads();
    for (int i = tid; i < kDpChunk; i += kDpThreads) sU[i] = b0 + i <= bmax ? __ldg(U + b0 + i) : -INFINITY;
    // sF[i] = prev[ybase + i], ybase = xbase - b0 - (kDpChunk - 1)
    const long long ybase = xbase - b0 - (kDpChunk - 1);
    for (int i = tid; i < kDpTile + kDpChunk; i += kDpThreads) {
      const long long y = ybase + i;
      sF[i] = (y >= plo && y <= phi) ? prev[y] : -INFINITY;
    }
    __syncthreads();
#pragma unroll 4
    for (int i = 0; i < kDpChunk; ++i) {
      const float u = sU[i];
      const int base = (kDpChunk - 1) - i + tid;  // index of x - b for r = 0
#pragma unroll
      for (int r = 0; r < kDpPer; ++r) {
        const float v = sF[base + r * kDpThreads] + u;
        if (v > best[r]) {
          best[r] = v;
          arg[r] = (int)(b0 + i);
        }
      }
    }
  }
#pragma unroll
  for (int r = 0; r < kDpPer; ++r) {
    const long long x = xbase + tid + (long long)r * kDpThreads;
    if (x <= hi) {
      next[x] = best[r];
      choice[x] = (unsigned short)arg[r];
    }
  }
}

// Walks back from x = B; also writes the optimum and the packed-row offsets of this sequence.
__global__ void dp_backtrack_kernel(const float* __restrict__ f, const unsigned short* __restrict__ choice,
                                    long long stride, long long B, int N, int w, long long row_base, int q,
                                    int32_t* __restrict__ budgets, int32_t* __restrict__ offsets,
                                    double* __restrict__ values) {
  if (threadIdx.x != 0 || blockIdx.x != 0) return;
  values[q] = (double)f[B];
  long long x = B;
  for (int h = N - 1; h >= 0; --h) {
    const int b = choice[(size_t)h * stride + x];
    budgets[(size_t)q * N + h] = b;
    x -= b;
  }
  if (q == 0) offsets[0] = 0;
  long long run = row_base;
  for (int h = 0; h < N; ++h) {
    run += budgets[(size_t)q * N + h] + w;
    offsets[(size_t)q * N + h + 1] = (int32_t)run;
  }
}

size_t align256x(size_t x) { return (x + 255) & ~(size_t)255; }

}  // namespace

size_t exact_workspace_bytes(const Dims& dm, int64_t max_budget) {
  const size_t cnt = (size_t)max_budget + 1;
  return 2 * align256x(cnt * sizeof(float)) + align256x((size_t)dm.N * cnt * sizeof(unsigned short));
}

cudaError_t launch_exact_allocate(const Dims& dm, const float* curves, const int64_t* budgets_host, int32_t* budgets,
                                  int32_t* offsets, double* values, void* ws, LaunchCtx& lc) {
  long long row_base = 0;
  for (int q = 0; q < dm.S; ++q) {
    const long long B = budgets_host[q];
    const size_t cnt = (size_t)B + 1;
    char* p = static_cast<char*>(ws);
    float* f0 = reinterpret_cast<float*>(p);
    float* f1 = reinterpret_cast<float*>(p + align256x(cnt * sizeof(float)));
    unsigned short* choice = reinterpret_cast<unsigned short*>(p + 2 * align256x(cnt * sizeof(float)));
    dp_init_kernel<<<(unsigned)((cnt + 255) / 256), 256, 0, lc.st>>>(f0, (long long)cnt);
    lc.mark("dp_init");
    long long plo = 0, phi = 0;
    float* prev = f0;
    float* next = f1;
    for (int h = 0; h < dm.N; ++h) {
      const long long lo = std::max(0LL, B - (long long)(dm.N - 1 - h) * dm.n);
      const long long hi = std::min(B, (long long)(h + 1) * dm.n);
      const unsigned blocks = (unsigned)((hi - lo + kDpTile) / kDpTile);
      dp_step_kernel<<<blocks, kDpThreads, 0, lc.st>>>(curves + (size_t)h * dm.P, prev, next, choice + (size_t)h * cnt,
                                                       dm.n, lo, hi, plo, phi);
      lc.mark("dp_step");
      plo = lo;
      phi = hi;
      float* t = prev;
      prev = next;
      next = t;
    }
    dp_backtrack_kernel<<<1, 32, 0, lc.st>>>(prev, choice, (long long)cnt, B, dm.N, dm.w, row_base, q, budgets, offsets,
                                             values);
    lc.mark("dp_backtrack");
    row_base += B + (long long)dm.N * dm.w;
  }
  return cudaGetLastError();
}

}  // namespace lukv
