// Offline profile and online lookup (paper Sec. 4.3).
//   profile_mean_kernel     Eq. "calibration_avg": the profile entry of (ratio, head) is the mean over
//                           the calibration queries of the optimal local ratio r* = 1 - b/n, where b is
//                           the head's budget in that query's solution of the relaxed problem.
//   profile_budget_kernel   "Lookup" and "Budgeting": r = profile row at the target ratio (linear
//                           interpolation between the two neighbouring grid rows), b = floor((1-r)*n).
//   offsets_scan_kernel     packed-row offsets of the resulting budgets.
// All ratio arithmetic is fp64 with explicit round-to-nearest operations (no contraction), because a
// floor follows it: the integer must not depend on how the compiler fuses the expression.
#include "common.cuh"

namespace lukv {
namespace {

constexpr int kProfileThreads = 256;

// budgets: [n_queries][count] with count = R*N; profile: [count].
__global__ void profile_mean_kernel(const int32_t* __restrict__ budgets, float* __restrict__ profile, int n_queries,
                                    long long count, int n) {
  const long long e = (long long)blockIdx.x * kProfileThreads + threadIdx.x;
  if (e >= count) return;
  const double dn = (double)n;
  double acc = 0.0;
  for (int i = 0; i < n_queries; ++i) {
    const double b = (double)budgets[(size_t)i * count + e];
    acc = __dadd_rn(acc, __dsub_rn(1.0, __ddiv_rn(b, dn)));
  }
  profile[e] = __double2float_rn(__ddiv_rn(acc, (double)n_queries));
}

struct LookupArgs {
  int row_lo[kLookupSeqPerLaunch];   // grid row at or below the target ratio
  int row_hi[kLookupSeqPerLaunch];   // the next row (== row_lo at the last grid point)
  double frac[kLookupSeqPerLaunch];  // position of the target between the two rows, in [0,1)
  int n[kLookupSeqPerLaunch];        // rankable positions of the sequence
  int floor_tok[kLookupSeqPerLaunch];  // its minimum retention in tokens
  int seq0;
};

// blockIdx.y = sequence of this launch, x covers the heads.
__global__ void profile_budget_kernel(const float* __restrict__ profile, LookupArgs args, int N,
                                      int32_t* __restrict__ budgets) {
  const int hid = blockIdx.x * kProfileThreads + threadIdx.x;
  if (hid >= N) return;
  const int i = blockIdx.y;
  const int n = args.n[i], floor_tok = args.floor_tok[i];
  const double r0 = (double)profile[(size_t)args.row_lo[i] * N + hid];
  const double r1 = (double)profile[(size_t)args.row_hi[i] * N + hid];
  const double r = __dadd_rn(r0, __dmul_rn(__dsub_rn(r1, r0), args.frac[i]));
  double b = floor(__dmul_rn(__dsub_rn(1.0, r), (double)n));
  b = b < 0.0 ? 0.0 : (b > (double)n ? (double)n : b);
  const int32_t bi = (int32_t)b;
  budgets[(size_t)(args.seq0 + i) * N + hid] = bi < floor_tok ? floor_tok : bi;  // minimum retention (App. E)
}

constexpr int kScanThreads = 1024;

// offsets[0] = 0, offsets[u+1] = sum_{v<=u} (budgets[v] + w).  One CTA; each thread owns a
// contiguous run of heads.
__global__ void __launch_bounds__(kScanThreads) offsets_scan_kernel(const int32_t* __restrict__ budgets,
                                                                    int32_t* __restrict__ offsets, int count, int w) {
  __shared__ long long warp_sums[kScanThreads / 32];
  const int tid = threadIdx.x;
  const int per = (count + kScanThreads - 1) / kScanThreads;
  const int u0 = min(count, tid * per), u1 = min(count, u0 + per);
  long long local = 0;
  for (int u = u0; u < u1; ++u) local += budgets[u] + w;
  long long incl = local;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const long long o = __shfl_up_sync(0xffffffffu, incl, off);
    if ((tid & 31) >= off) incl += o;
  }
  if ((tid & 31) == 31) warp_sums[tid >> 5] = incl;
  __syncthreads();
  long long run = incl - local;
  for (int wv = 0; wv < (tid >> 5); ++wv) run += warp_sums[wv];
  if (tid == 0) offsets[0] = 0;
  for (int u = u0; u < u1; ++u) {
    run += budgets[u] + w;
    offsets[u + 1] = (int32_t)run;
  }
}

}  // namespace

cudaError_t launch_profile_mean(const int32_t* budgets, float* profile, int n_queries, int64_t count, int n,
                                LaunchCtx& lc) {
  const unsigned blocks = (unsigned)((count + kProfileThreads - 1) / kProfileThreads);
  profile_mean_kernel<<<blocks, kProfileThreads, 0, lc.st>>>(budgets, profile, n_queries, (long long)count, n);
  lc.mark("profile_mean");
  return cudaGetLastError();
}

cudaError_t launch_profile_budgets(const float* profile, const int* row_lo, const int* row_hi, const double* frac,
                                   const Dims& dm, int32_t* budgets, int32_t* offsets, LaunchCtx& lc) {
  const int S = dm.S, N = dm.N, w = dm.w;
  for (int q0 = 0; q0 < S; q0 += kLookupSeqPerLaunch) {
    LookupArgs args;
    const int cnt = S - q0 < kLookupSeqPerLaunch ? S - q0 : kLookupSeqPerLaunch;
    for (int i = 0; i < kLookupSeqPerLaunch; ++i) {
      args.row_lo[i] = i < cnt ? row_lo[q0 + i] : 0;
      args.row_hi[i] = i < cnt ? row_hi[q0 + i] : 0;
      args.frac[i] = i < cnt ? frac[q0 + i] : 0.0;
      args.n[i] = i < cnt ? seq_rankable(dm, q0 + i) : 0;
      args.floor_tok[i] = i < cnt ? seq_floor_tokens(dm, q0 + i) : 0;
    }
    args.seq0 = q0;
    profile_budget_kernel<<<dim3((N + kProfileThreads - 1) / kProfileThreads, cnt), kProfileThreads, 0, lc.st>>>(
        profile, args, N, budgets);
    lc.mark("profile_budget");
  }
  offsets_scan_kernel<<<1, kScanThreads, 0, lc.st>>>(budgets, offsets, S * N, w);
  lc.mark("offsets_scan");
  return cudaGetLastError();
}

}  // namespace lukv
