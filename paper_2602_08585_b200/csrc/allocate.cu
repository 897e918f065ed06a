// Stage (b): global head-level budget allocation (paper Sec. 4.2, App. A.2).
//   hull_kernel    PAVA projection of every head's curve increments onto a non-increasing,
//                  non-negative sequence (Eq. "marginal_gain"), fp64 with explicit
//                  round-to-nearest operations, gains rounded once to fp32.
//   greedy_kernel  the marginal-utility greedy, computed as a weighted radix select: the
//                  greedy consumes curve segments in the order (gain desc, k asc, hid asc);
//                  the kernel finds the segment at which the budget runs out and gives
//                  every head the capacity of its segments before that point.
#include "common.cuh"

namespace lukv {
namespace {

// ---- hull ----------------------------------------------------------------------------

// mean(a/b) <= mean(c/d) decided exactly as the comparison of the two correctly rounded
// fp64 quotients (b, d > 0).  The products decide whenever they are clearly apart (then the
// rounded quotients are ordered the same way); otherwise the quotients themselves are
// compared.
__device__ __forceinline__ bool mean_le(double a, double b, double c, double d) {
  const double p1 = __dmul_rn(a, d), p2 = __dmul_rn(c, b);
  const double diff = __dsub_rn(p1, p2);
  const double tol = fmax(fabs(p1), fabs(p2)) * 9.094947017729282e-13;  // 2^-40
  if (diff < -tol) return true;
  if (diff > tol) return false;
  return __ddiv_rn(a, b) <= __ddiv_rn(c, d);
}

// One thread per head; a block stages `hb` heads in shared memory, interleaved by head so
// that every thread stays in its own bank.  Stack entries are block start points; a
// block's end is the next entry's start.
__global__ void hull_kernel(const float* __restrict__ curves, float* __restrict__ gains, int N, int P, int hb) {
  extern __shared__ __align__(16) unsigned char hull_smem[];
  float* Us = reinterpret_cast<float*>(hull_smem);   // [P][hb]; overwritten by the gains
  int* Ls = reinterpret_cast<int*>(Us + (size_t)P * hb);  // [P][hb]
  const int hid0 = blockIdx.x * hb;
  const int heads_here = min(hb, N - hid0);
  for (int i = threadIdx.x; i < heads_here * P; i += blockDim.x) {
    const int h = i / P, p = i % P;
    Us[p * hb + h] = curves[(size_t)(hid0 + h) * P + p];
  }
  __syncthreads();
  const int h = threadIdx.x;
  if (h < heads_here) {
    int sp = 0;
    for (int k = 0; k + 1 < P; ++k) {
      int cur_l = k;
      const int cur_r = k + 1;
      const double u_r = (double)Us[cur_r * hb + h];
      double cur_num = __dsub_rn(u_r, (double)Us[cur_l * hb + h]);
      double cur_den = 1.0;
      while (sp > 0) {
        const int top_l = Ls[(sp - 1) * hb + h];
        const double top_num = __dsub_rn((double)Us[cur_l * hb + h], (double)Us[top_l * hb + h]);
        const double top_den = (double)(cur_l - top_l);
        if (!mean_le(top_num, top_den, cur_num, cur_den)) break;
        cur_l = top_l;
        --sp;
        cur_num = __dsub_rn(u_r, (double)Us[cur_l * hb + h]);
        cur_den = (double)(cur_r - cur_l);
      }
      Ls[sp * hb + h] = cur_l;
      ++sp;
    }
    for (int i = 0; i < sp; ++i) {
      const int l = Ls[i * hb + h];
      const int r = (i + 1 < sp) ? Ls[(i + 1) * hb + h] : P - 1;
      const double mean = __ddiv_rn(__dsub_rn((double)Us[r * hb + h], (double)Us[l * hb + h]), (double)(r - l));
      const float g = __double2float_rn(mean > 0.0 ? mean : 0.0);
      for (int k = l; k < r; ++k) Us[k * hb + h] = g;  // U[l..r-1] are no longer needed
    }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < heads_here * (P - 1); i += blockDim.x) {
    const int hh = i / (P - 1), kk = i % (P - 1);
    gains[(size_t)(hid0 + hh) * (P - 1) + kk] = Us[kk * hb + hh];
  }
}

// ---- greedy --------------------------------------------------------------------------

constexpr int kGreedyThreads = 256;
constexpr int kSeqPerLaunch = 32;

struct GreedyArgs {
  long long budget[kSeqPerLaunch];    // B_q
  long long row_base[kSeqPerLaunch];  // packed rows before sequence q
  int seq0;                           // first sequence of this launch
};

// Sort key of segment (hid,k): ascending key order == greedy consumption order.
__device__ __forceinline__ unsigned long long seg_key(float gain, unsigned k, unsigned hid, unsigned N) {
  return ((unsigned long long)(~__float_as_uint(gain)) << 32) | (unsigned long long)(k * N + hid);
}

__device__ __forceinline__ long long capsum(int c, int seg, int n) {  // tokens in segments [0,c)
  const long long t = (long long)c * seg;
  return t < n ? t : (long long)n;
}

// One CTA per sequence.  Within a head the keys increase with k (gains are non-increasing),
// so the segments of a head that still match the key prefix form a range [lo,hi); segments
// before lo are already bought.  Each of the 8 passes histograms the next key byte of the
// active segments weighted by capacity, picks the byte at which the remaining budget runs
// out and narrows every head's range to it.  Keys are unique, so one segment remains: the
// partially bought one.
__global__ void __launch_bounds__(kGreedyThreads) greedy_kernel(const float* __restrict__ gains, GreedyArgs args,
                                                                int32_t* __restrict__ budgets,
                                                                int32_t* __restrict__ offsets, int N, int P, int seg,
                                                                int nseg, int n, int w) {
  extern __shared__ __align__(16) unsigned char greedy_smem[];
  int* lo = reinterpret_cast<int*>(greedy_smem);  // [N]
  int* hi = lo + N;                               // [N]
  __shared__ unsigned long long hist[256];
  __shared__ long long sh_remaining;
  __shared__ int sh_digit, sh_all_taken;
  __shared__ long long warp_sums[kGreedyThreads / 32];

  const int q = args.seq0 + blockIdx.x;
  const int tid = threadIdx.x;
  const int G1 = P - 1;
  for (int h = tid; h < N; h += kGreedyThreads) {
    lo[h] = 0;
    hi[h] = nseg;
  }
  if (tid == 0) {
    sh_remaining = args.budget[blockIdx.x];
    sh_all_taken = 0;
  }
  __syncthreads();

  for (int pass = 0; pass < 8; ++pass) {
    const int shift = 56 - 8 * pass;
    hist[tid] = 0ull;  // kGreedyThreads == 256 bins
    __syncthreads();
    for (int h = tid; h < N; h += kGreedyThreads) {
      const int l = lo[h], r = hi[h];
      if (l >= r) continue;
      const float* g = gains + (size_t)h * G1;
      int run_start = l;
      unsigned run_digit = (unsigned)(seg_key(__ldg(g + l), l, h, N) >> shift) & 255u;
      for (int k = l + 1; k < r; ++k) {
        const unsigned dgt = (unsigned)(seg_key(__ldg(g + k), k, h, N) >> shift) & 255u;
        if (dgt != run_digit) {
          atomicAdd(&hist[run_digit], (unsigned long long)(capsum(k, seg, n) - capsum(run_start, seg, n)));
          run_start = k;
          run_digit = dgt;
        }
      }
      atomicAdd(&hist[run_digit], (unsigned long long)(capsum(r, seg, n) - capsum(run_start, seg, n)));
    }
    __syncthreads();
    if (tid < 32) {
      // lane owns bins [8*lane, 8*lane+8); find the first bin whose running total exceeds
      // the remaining budget
      const long long R = sh_remaining;
      long long mine = 0;
#pragma unroll
      for (int b = 0; b < 8; ++b) mine += (long long)hist[tid * 8 + b];
      long long incl = mine;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const long long o = __shfl_up_sync(0xffffffffu, incl, off);
        if (tid >= off) incl += o;
      }
      const long long excl = incl - mine;
      const long long total = __shfl_sync(0xffffffffu, incl, 31);
      if (total <= R) {
        if (tid == 0) {
          sh_all_taken = 1;
          sh_remaining = R - total;
        }
      } else if (excl <= R && R < incl) {
        long long run = excl;
        for (int b = 0; b < 8; ++b) {
          const long long hval = (long long)hist[tid * 8 + b];
          if (run + hval > R) {
            sh_digit = tid * 8 + b;
            sh_remaining = R - run;
            break;
          }
          run += hval;
        }
      }
    }
    __syncthreads();
    if (sh_all_taken) {
      for (int h = tid; h < N; h += kGreedyThreads) lo[h] = hi[h];
      break;
    }
    const unsigned D = (unsigned)sh_digit;
    for (int h = tid; h < N; h += kGreedyThreads) {
      int l = lo[h], r = hi[h];
      if (l >= r) continue;
      const float* g = gains + (size_t)h * G1;
      // digits are non-decreasing in k: binary searches for the first digit >= D and > D
      int a = l, b = r;
      while (a < b) {
        const int mid = (a + b) >> 1;
        const unsigned dgt = (unsigned)(seg_key(__ldg(g + mid), mid, h, N) >> shift) & 255u;
        if (dgt < D) a = mid + 1; else b = mid;
      }
      const int nl = a;
      b = r;
      while (a < b) {
        const int mid = (a + b) >> 1;
        const unsigned dgt = (unsigned)(seg_key(__ldg(g + mid), mid, h, N) >> shift) & 255u;
        if (dgt <= D) a = mid + 1; else b = mid;
      }
      lo[h] = nl;
      hi[h] = a;
    }
    __syncthreads();
  }
  __syncthreads();

  // budgets, then offsets = row_base + exclusive scan of (budget + w)
  const long long R = sh_remaining;
  const int per = (N + kGreedyThreads - 1) / kGreedyThreads;
  const int h_begin = min(N, tid * per), h_end = min(N, h_begin + per);
  long long local = 0;
  for (int h = h_begin; h < h_end; ++h) {
    long long b = capsum(lo[h], seg, n);
    if (hi[h] > lo[h]) b += R;  // the one partially bought segment
    lo[h] = (int)b;
    local += b + w;
  }
  long long incl = local;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const long long o = __shfl_up_sync(0xffffffffu, incl, off);
    if ((tid & 31) >= off) incl += o;
  }
  if ((tid & 31) == 31) warp_sums[tid >> 5] = incl;
  __syncthreads();
  long long before = 0;
  for (int wv = 0; wv < (tid >> 5); ++wv) before += warp_sums[wv];
  long long run = args.row_base[blockIdx.x] + before + incl - local;
  if (q == 0 && tid == 0) offsets[0] = 0;
  for (int h = h_begin; h < h_end; ++h) {
    budgets[(size_t)q * N + h] = lo[h];
    run += lo[h] + w;
    offsets[(size_t)q * N + h + 1] = (int32_t)run;
  }
}

}  // namespace

cudaError_t launch_allocate(const Dims& dm, const float* curves, const int64_t* budgets_host, float* gains,
                            int32_t* budgets, int32_t* offsets, LaunchCtx& lc) {
  cudaStream_t st = lc.st;
  // hull: as many heads per block as fit in ~200 KB of shared memory, at most 32
  int hb = (int)((200u * 1024u) / ((size_t)dm.P * 8u));
  hb = hb > 32 ? 32 : (hb < 1 ? 1 : hb);
  const size_t hull_smem = (size_t)dm.P * hb * 8;
  cudaError_t e;
  if ((e = cudaFuncSetAttribute(hull_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)hull_smem)) != cudaSuccess)
    return e;
  hull_kernel<<<(dm.N + hb - 1) / hb, 128, hull_smem, st>>>(curves, gains, dm.N, dm.P, hb);
  lc.mark("hull");

  const size_t greedy_smem = (size_t)dm.N * 2 * sizeof(int);
  if ((e = cudaFuncSetAttribute(greedy_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)greedy_smem)) != cudaSuccess)
    return e;
  long long base = 0;
  for (int q0 = 0; q0 < dm.S; q0 += kSeqPerLaunch) {
    GreedyArgs args;
    const int cnt = dm.S - q0 < kSeqPerLaunch ? dm.S - q0 : kSeqPerLaunch;
    for (int i = 0; i < kSeqPerLaunch; ++i) {
      args.budget[i] = 0;
      args.row_base[i] = 0;
    }
    for (int i = 0; i < cnt; ++i) {
      args.budget[i] = budgets_host[q0 + i];
      args.row_base[i] = base;
      base += budgets_host[q0 + i] + (long long)dm.N * dm.w;
    }
    args.seq0 = q0;
    greedy_kernel<<<cnt, kGreedyThreads, greedy_smem, st>>>(gains, args, budgets, offsets, dm.N, dm.P, dm.seg, dm.nseg,
                                                            dm.n, dm.w);
    lc.mark("greedy");
  }
  return cudaGetLastError();
}

}  // namespace lukv
