// Stage (b): global head-level budget allocation (paper Sec. 4.2, App. A.2).
//   hull_kernel    PAVA projection of every head's curve increments onto a non-increasing,
//                  non-negative sequence (Eq. "marginal_gain"); merge decisions equal to the
//                  comparison of fp64 block means, gains fp64 with explicit round-to-nearest
//                  operations, rounded once to fp32.
//   greedy_kernel  the marginal-utility greedy, computed as a weighted selection: the greedy
//                  consumes curve segments in the order (gain desc, k asc, hid asc); the
//                  kernel finds the segment at which the budget runs out by bisection over
//                  the key bits (one binary search per head and bit) and gives every head
//                  the capacity of its segments before that point.
#include "common.cuh"

namespace lukv {
namespace {

// ---- hull ----------------------------------------------------------------------------

// mean of block 1 <= mean of block 2, where a block's mean is (its curve rise) / (its length) and
// the rises are differences of two fp32 curve values: decided exactly as the comparison of the two
// correctly rounded fp64 quotients.  Three tiers, cheapest first (the fp64 pipe is slow, and the
// walk below is one dependent chain):
//   fp32 cross products, when they are further apart than fp32 rounding can explain;
//   fp64 cross products, when they are clearly apart;
//   the fp64 quotients themselves.
// Block 1 rises from u_l1 to u_r1 over len1 points, block 2 from u_l2 to u_r2 over len2.
__device__ __forceinline__ bool mean_le(float u_l1, float u_r1, int len1, float u_l2, float u_r2, int len2) {
  const float fa = u_r1 - u_l1, fb = (float)len1, fc = u_r2 - u_l2, fd = (float)len2;
  const float q1 = fa * fd, q2 = fc * fb;
  const float ftol = 4e-7f * fmaxf(fabsf(q1), fabsf(q2));  // each product carries two roundings of 2^-24
  if (q1 < q2 - ftol) return true;
  if (q1 > q2 + ftol) return false;
  const double a = __dsub_rn((double)u_r1, (double)u_l1), b = (double)len1;
  const double c = __dsub_rn((double)u_r2, (double)u_l2), d = (double)len2;
  const double p1 = __dmul_rn(a, d), p2 = __dmul_rn(c, b);
  const double diff = __dsub_rn(p1, p2);
  const double tol = fmax(fabs(p1), fabs(p2)) * 9.094947017729282e-13;  // 2^-40
  if (diff < -tol) return true;
  if (diff > tol) return false;
  return __ddiv_rn(a, b) <= __ddiv_rn(c, d);
}

// Shared memory of one warp of the hull kernel: the stack of block starts, [P] 16-bit indices.
__host__ __device__ inline size_t hull_bytes_per_warp(int P) { return ((size_t)P * 2 + 15) & ~(size_t)15; }

// One warp per curve.  Lane 0 runs the pool-adjacent-violators stack (the sequence of merge
// decisions is the algorithm; it is serial by nature).  The walk is one dependent chain, so what it
// touches per step is kept short: the curve values at the starts of the top block and of the
// current block live in registers, the next curve point is requested one step ahead (the curve is
// read through L1: the walk streams it, a pop re-reads a point that was read not long before), and
// the stack of block starts is the only thing in shared memory (2 bytes per point, so that many
// warps fit an SM when thousands of long curves are projected at once).  The other lanes join for
// the output: one block of the result per lane at a time.
// Stack entries are block start points; a block's end is the next entry's start.
__global__ void hull_kernel(const float* __restrict__ curves, float* __restrict__ gains, int N, int P) {
  extern __shared__ __align__(16) unsigned char hull_smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int warps = blockDim.x >> 5;
  const int hid = blockIdx.x * warps + warp;
  if (hid >= N) return;  // whole warps leave together; only __syncwarp is used below
  const float* U = curves + (size_t)hid * P;
  unsigned short* Ls = reinterpret_cast<unsigned short*>(hull_smem + (size_t)warp * hull_bytes_per_warp(P));
  int sp = 0;
  if (lane == 0) {
    int top_l = 0;        // start of the block on top of the stack; it ends where the current block starts
    float u_top = 0.f;    // U[top_l]
    float u_k = __ldg(U), u_next = __ldg(U + 1);
    for (int k = 0; k + 1 < P; ++k) {
      const float u_ahead = k + 2 < P ? __ldg(U + k + 2) : 0.f;  // for the next step
      int cur_l = k;
      float u_cur = u_k;  // U[cur_l]
      while (sp > 0 && mean_le(u_top, u_cur, cur_l - top_l, u_cur, u_next, k + 1 - cur_l)) {
        cur_l = top_l;
        u_cur = u_top;
        --sp;
        if (sp > 0) {
          top_l = Ls[sp - 1];
          u_top = __ldg(U + top_l);
        }
      }
      Ls[sp++] = (unsigned short)cur_l;
      top_l = cur_l;
      u_top = u_cur;
      u_k = u_next;
      u_next = u_ahead;
    }
  }
  sp = __shfl_sync(0xffffffffu, sp, 0);
  __syncwarp();
  float* out = gains + (size_t)hid * (P - 1);
  for (int i = lane; i < sp; i += 32) {
    const int l = Ls[i];
    const int r = (i + 1 < sp) ? (int)Ls[i + 1] : P - 1;
    const double mean = __ddiv_rn(__dsub_rn((double)__ldg(U + r), (double)__ldg(U + l)), (double)(r - l));
    const float g = __double2float_rn(mean > 0.0 ? mean : 0.0);
    for (int k = l; k < r; ++k) out[k] = g;
  }
}

// ---- greedy --------------------------------------------------------------------------

constexpr int kGreedyMaxThreads = 1024;
constexpr int kSeqPerLaunch = 32;

struct GreedyArgs {
  long long budget[kSeqPerLaunch];    // B_q
  long long row_base[kSeqPerLaunch];  // packed rows before sequence q
  int T[kSeqPerLaunch];               // context length of sequence q (the curve grid is T/(P-1) tokens per segment)
  int floor_tok[kSeqPerLaunch];       // tokens every head of sequence q keeps at least
  int seq0;                           // first sequence of this launch
};

struct SetStride {
  size_t gains, budgets, offsets;  // elements between consecutive curve sets
};

// Sort key of segment (hid,k): ascending key order == greedy consumption order.
__device__ __forceinline__ unsigned long long seg_key(float gain, unsigned k, unsigned hid, unsigned N) {
  return ((unsigned long long)(~__float_as_uint(gain)) << 32) | (unsigned long long)(k * N + hid);
}

// Tokens for sale in segments [0,c) of a head whose first `floor_tok` tokens were handed to it up
// front (the minimum retention of App. E; 0 = none).
__device__ __forceinline__ long long capsum(int c, int seg, int n, int floor_tok) {
  long long t = (long long)c * seg;
  t = (t < n ? t : (long long)n) - floor_tok;
  return t > 0 ? t : 0;
}

// Block-wide sum; every thread gets the result.  `buf` holds one value per warp.  One barrier per
// call is enough only if consecutive calls use different buffers: the caller alternates between two.
__device__ __forceinline__ long long block_sum_ll(long long v, long long* buf) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
  if ((threadIdx.x & 31) == 0) buf[threadIdx.x >> 5] = v;
  __syncthreads();
  long long total = 0;
  const int warps = blockDim.x >> 5;
  for (int x = 0; x < warps; ++x) total += buf[x];
  return total;
}

// One CTA per (sequence, curve set), one thread per head (a CTA of fewer threads than heads loops).
// The greedy buys segments in ascending key order until the budget is spent; the kernel finds the
// key at which that happens by bisection over the 64 key bits.  Within a head the keys increase
// with k (gains are non-increasing), so the segments of a head that share the key prefix fixed so
// far form a range [lo,hi), segments before lo are bought, and inside the range the next key bit is
// 0 up to some index and 1 from there on: one binary search per head and bit finds that index (no
// search at all when the range's two ends agree), the capacities below it are summed over the
// heads, and the budget decides which half holds the cut.  Keys are unique, so after the last bit
// one segment remains: the partially bought one.
//
// blockIdx.y selects one of several independent curve sets (the calibration queries of the
// offline profile, which share the budgets): set i reads gains + i*set.gains, writes
// budgets + i*set.budgets and offsets + i*set.offsets.  The hot path launches one set.
__global__ void __launch_bounds__(kGreedyMaxThreads) greedy_kernel(const float* __restrict__ gains, GreedyArgs args,
                                                                   int32_t* __restrict__ budgets,
                                                                   int32_t* __restrict__ offsets, SetStride set,
                                                                   int N, int P, int w) {
  // the sequence's own grid: n rankable positions, seg tokens per curve segment, nseg segments with capacity
  const int n = args.T[blockIdx.x] - w, seg = args.T[blockIdx.x] / (P - 1), nseg = (n + seg - 1) / seg;
  const int floor_tok = args.floor_tok[blockIdx.x];
  gains += (size_t)blockIdx.y * set.gains;
  budgets += (size_t)blockIdx.y * set.budgets;
  offsets += (size_t)blockIdx.y * set.offsets;
  extern __shared__ __align__(16) unsigned char greedy_smem[];
  int* lo = reinterpret_cast<int*>(greedy_smem);  // [N]
  int* hi = lo + N;                               // [N]
  int* mid = hi + N;                              // [N]
  __shared__ long long sum_buf[2][kGreedyMaxThreads / 32];
  __shared__ long long warp_sums[kGreedyMaxThreads / 32];

  const int q = args.seq0 + blockIdx.x;
  const int tid = threadIdx.x, nthr = blockDim.x;
  const int G1 = P - 1;
  long long R = args.budget[blockIdx.x] - (long long)N * floor_tok;  // the floor is spent before the greedy
  const bool all_taken = (long long)N * (n - floor_tok) <= R;
  for (int h = tid; h < N; h += nthr) {
    lo[h] = all_taken ? nseg : 0;
    hi[h] = nseg;
  }
  // (each thread only ever touches the heads it owns, so lo/hi/mid need no barrier of their own)
  if (!all_taken) {
    // the low key word is k*N + hid < N*(P-1): its bits from idx_bits up are zero in every key, a pass over
    // them would change nothing
    int idx_bits = 0;
    while (idx_bits < 32 && ((unsigned long long)N * (unsigned)G1) >> idx_bits) ++idx_bits;
    int round = 0;  // executed iterations: selects the sum buffer (the skipped bits must not count)
    for (int bit = 63; bit >= 0; --bit) {
      if (bit < 32 && bit >= idx_bits) continue;
      long long local = 0;
      for (int h = tid; h < N; h += nthr) {
        const int l = lo[h], r = hi[h];
        int m = l;
        if (l < r) {
          const float* g = gains + (size_t)h * G1;
          auto bit_at = [&](int k) { return (int)((seg_key(__ldg(g + k), k, h, N) >> bit) & 1ull); };
          if (bit_at(l)) {
            m = l;
          } else if (!bit_at(r - 1)) {
            m = r;
          } else {
            int a = l, b = r - 1;  // bit(a) == 0, bit(b) == 1
            while (b - a > 1) {
              const int c = (a + b) >> 1;
              if (bit_at(c)) b = c; else a = c;
            }
            m = b;
          }
        }
        mid[h] = m;
        local += capsum(m, seg, n, floor_tok) - capsum(l, seg, n, floor_tok);
      }
      const long long tokens0 = block_sum_ll(local, sum_buf[round++ & 1]);
      if (tokens0 > R) {
        for (int h = tid; h < N; h += nthr) hi[h] = mid[h];
      } else {
        R -= tokens0;
        for (int h = tid; h < N; h += nthr) lo[h] = mid[h];
      }
    }
  }

  // budgets, then offsets = row_base + exclusive scan of (budget + w)
  const int per = (N + nthr - 1) / nthr;
  const int h_begin = min(N, tid * per), h_end = min(N, h_begin + per);
  __syncthreads();  // the scan below re-partitions the heads over the threads
  long long local = 0;
  for (int h = h_begin; h < h_end; ++h) {
    long long b = floor_tok + capsum(lo[h], seg, n, floor_tok);
    if (hi[h] > lo[h]) b += R;  // the one partially bought segment
    mid[h] = (int)b;
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
    budgets[(size_t)q * N + h] = mid[h];
    run += mid[h] + w;
    offsets[(size_t)q * N + h + 1] = (int32_t)run;
  }
}

}  // namespace

cudaError_t launch_hull(const float* curves, float* gains, int64_t n_curves, int P, LaunchCtx& lc) {
  // one warp per curve; few curves: small blocks, so that they spread over the SMs (each walk is a
  // latency-bound chain); many curves: up to 8 warps per block
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  int hw = (int)((n_curves + sms - 1) / sms);
  hw = hw > 8 ? 8 : (hw < 1 ? 1 : hw);
  const size_t hull_smem = hull_bytes_per_warp(P) * hw;
  cudaError_t e;
  if ((e = cudaFuncSetAttribute(hull_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)hull_smem)) != cudaSuccess)
    return e;
  hull_kernel<<<(unsigned)((n_curves + hw - 1) / hw), hw * 32, hull_smem, lc.st>>>(curves, gains, (int)n_curves, P);
  lc.mark("hull");
  return cudaGetLastError();
}

cudaError_t launch_greedy(const Dims& dm, const float* gains, const int64_t* budgets_host, int32_t* budgets,
                          int32_t* offsets, int n_sets, LaunchCtx& lc) {
  cudaError_t e;
  const size_t greedy_smem = (size_t)dm.N * 3 * sizeof(int);
  int threads = (dm.N + 31) & ~31;  // one thread per head, whole warps
  if (threads > kGreedyMaxThreads) threads = kGreedyMaxThreads;
  if ((e = cudaFuncSetAttribute(greedy_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)greedy_smem)) != cudaSuccess)
    return e;
  SetStride set;
  set.gains = (size_t)dm.N * (dm.P - 1);
  set.budgets = (size_t)dm.S * dm.N;
  set.offsets = (size_t)dm.S * dm.N + 1;
  long long base = 0;
  for (int q0 = 0; q0 < dm.S; q0 += kSeqPerLaunch) {
    GreedyArgs args;
    const int cnt = dm.S - q0 < kSeqPerLaunch ? dm.S - q0 : kSeqPerLaunch;
    for (int i = 0; i < kSeqPerLaunch; ++i) {
      args.budget[i] = 0;
      args.row_base[i] = 0;
      args.T[i] = dm.T;
      args.floor_tok[i] = dm.floor_tok;
    }
    for (int i = 0; i < cnt; ++i) {
      args.budget[i] = budgets_host[q0 + i];
      args.row_base[i] = base;
      if (dm.seq_T) {
        args.T[i] = dm.seq_T[q0 + i];
        args.floor_tok[i] = seq_floor_tokens(dm, q0 + i);
      }
      base += budgets_host[q0 + i] + (long long)dm.N * dm.w;
    }
    args.seq0 = q0;
    greedy_kernel<<<dim3(cnt, n_sets), threads, greedy_smem, lc.st>>>(gains, args, budgets, offsets, set, dm.N, dm.P,
                                                                      dm.w);
    lc.mark("greedy");
  }
  return cudaGetLastError();
}

cudaError_t launch_allocate(const Dims& dm, const float* curves, const int64_t* budgets_host, float* gains,
                            int32_t* budgets, int32_t* offsets, LaunchCtx& lc) {
  cudaError_t e = launch_hull(curves, gains, dm.N, dm.P, lc);
  if (e != cudaSuccess) return e;
  return launch_greedy(dm, gains, budgets_host, budgets, offsets, 1, lc);
}

}  // namespace lukv
