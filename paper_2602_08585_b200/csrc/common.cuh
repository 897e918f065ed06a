// Internal declarations shared by the translation units of liblukv.so.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stddef.h>
#include <stdint.h>

#include "lukv.h"

namespace lukv {

// Problem sizes derived once from lukv_params_t (validated by the API layer).
struct Dims {
  int S, L, H, G, d, T, w, kp, dtype, P;
  int N;        // heads per sequence
  int n;        // rankable positions per head
  int M;        // score rows per head = G*w
  int seg;      // tokens per curve segment s = T/(P-1)
  int nseg;     // curve segments with non-zero capacity = ceil(n/seg)
  float scale_log2;  // softmax scale * log2(e): logits are kept in the exp2 domain
  int n_sink;        // leading positions that rank first in the selection
  int floor_tok;     // tokens every head keeps at least: ceil(min_keep * n)
  // Sequences of different lengths in one call: seq_T[q] (HOST, S entries) is the context length of sequence q;
  // T, n and the tensor strides then describe the longest one.  nullptr: every sequence has length T.
  const int32_t* seq_T = nullptr;
  float min_keep = 0.f;  // as given (the per-sequence floors of a ragged call are derived from it)
  bool keydiff = false;  // stage (a) is the KeyDiff metric (keys only, no pooling)
  int64_t heads() const { return (int64_t)S * N; }
  size_t esize() const { return dtype == LUKV_DTYPE_BF16 ? 2 : 4; }
};

// Workspace carve-up (all offsets 256-byte aligned).
struct Workspace {
  float* raw;        // [S*N][n]   un-pooled scores
  float* pooled;     // [S*N][n]   pooled scores (fused path)
  float* stats;      // partial (reference, sum-exp) per row: [S*N][chunks][M][2] (FP32-pipe scorer) or
                     // [S*N][items][256][2] (tensor-core scorer)
  float* lse;        // [S*N][M]   row log-sum-exp in the exp2 domain
  float* gains;      // [N][P-1]   hull gains
  int* head_flags;   // tensor-core scorer: [S*N] items delivered per head, then the (lse, tag) rows
  size_t bytes;
};

int score_chunks(const Dims& dm);                       // key chunks per head of the SIMT scorer
size_t score_tc_stats_bytes(const Dims& dm);            // pass-1 partials of the two-sweep tensor-core scorer
size_t score_tc_flag_bytes(const Dims& dm);             // zero-initialised block: [heads] counters, then the (lse, tag) rows
size_t score_tc_lse_offset(const Dims& dm);             // offset of the (lse, tag) rows inside that block
void score_test_hooks(uint32_t* spin_limit, int* drop_item);  // environment hooks for the timeout tests
// Single-sweep tensor-core scorer: takes a shape if a head's work items fit kOnePassMaxItems CTAs.
constexpr int kOnePassMaxItems = 128;
bool score_onepass_eligible(const Dims& dm);
size_t score_onepass_stats_bytes(const Dims& dm);       // its per-(row, key tile) partials; 0 if not eligible
Workspace carve_workspace(const Dims& dm, void* base);  // base may be null (size query)

// Heads per sequence the greedy kernel can hold: 12 bytes of shared memory each, 227 KB per CTA
// less its static arrays.
constexpr int kGreedyMaxHeads = 18944;

// Most sequences a call with per-sequence context lengths takes: their lengths travel by value in the launch
// arguments of the kernels.
constexpr int kMaxRaggedSeqs = 64;
struct SeqLens {
  int T[kMaxRaggedSeqs];
};

// Rankable positions and minimum retention (tokens) of sequence q: the call's own when all sequences have one
// length, else from its length (the floor is ceil(min_keep * n) in fp64, as in the uniform case).
inline int seq_rankable(const Dims& dm, int q) { return dm.seq_T ? dm.seq_T[q] - dm.w : dm.n; }
inline int seq_floor_tokens(const Dims& dm, int q) {
  if (!dm.seq_T) return dm.floor_tok;
  const int n = dm.seq_T[q] - dm.w;
  const double fl = ceil((double)dm.min_keep * (double)n);
  return fl < 0.0 ? 0 : (fl > (double)n ? n : (int)fl);
}

// Launch bookkeeping: counts the kernels a call enqueues and, when a timeline is attached
// (profiling entry point only), records a CUDA event after each of them.
struct LaunchCtx {
  cudaStream_t st = nullptr;
  int launches = 0;
  cudaEvent_t* events = nullptr;  // [max_events + 1]; events[0] is recorded by the caller
  const char** names = nullptr;   // [max_events]
  int max_events = 0;
  void mark(const char* name) {
    if (events && launches < max_events) {
      names[launches] = name;
      cudaEventRecord(events[launches + 1], st);
    }
    ++launches;
  }
};

// Heads [h0, h0+nh) of the S*N heads of a call (the stages after allocation work head by head).
struct HeadRange {
  int h0, nh;
};

// Launchers.  Each returns cudaGetLastError() after its launches.
cudaError_t launch_score_simt(const Dims& dm, const void* q, const void* k, const Workspace& ws, LaunchCtx& lc);
// Folds per-chunk (max, sum-exp) partials [heads][chunks][M][2] into lse[heads][M] (exp2 domain).
cudaError_t launch_lse(const Dims& dm, const float* stats, float* lse, int chunks, LaunchCtx& lc);
// Tensor-core scorer (bf16, head_dim 128).  dev_status may be null.
bool score_tc_supported(const Dims& dm);
// clear_flags: zero the scorer's counters and (lse, tag) rows first (once per call, before the first range)
// spare_sms: SMs the persistent grid leaves to kernels of other streams
cudaError_t launch_score_tc(const Dims& dm, const void* q, const void* k, const Workspace& ws, int32_t* dev_status,
                            HeadRange hr, bool clear_flags, int spare_sms, LaunchCtx& lc);
// The single-sweep kernel alone; cudaErrorNotSupported (nothing launched) if the device has too few SMs for the shape.
cudaError_t launch_score_onepass(const Dims& dm, const void* q, const void* k, const Workspace& ws,
                                 int32_t* dev_status, HeadRange hr, bool clear_flags, int spare_sms, LaunchCtx& lc);
cudaError_t launch_pool(const Dims& dm, const float* raw, float* pooled, HeadRange hr, LaunchCtx& lc);
cudaError_t launch_allocate(const Dims& dm, const float* curves, const int64_t* budgets_host, float* gains,
                            int32_t* budgets, int32_t* offsets, LaunchCtx& lc);
// The two halves of launch_allocate.  launch_hull treats its input as n_curves independent curves;
// launch_greedy solves n_sets curve sets (gains [n_sets][N][P-1]) for the same dm.S budgets and
// writes budgets [n_sets][S][N] and offsets [n_sets][S*N+1].
cudaError_t launch_hull(const float* curves, float* gains, int64_t n_curves, int P, LaunchCtx& lc);
cudaError_t launch_greedy(const Dims& dm, const float* gains, const int64_t* budgets_host, int32_t* budgets,
                          int32_t* offsets, int n_sets, LaunchCtx& lc);
// Offline profile (mean of the local ratios) and online lookup + budgeting.
cudaError_t launch_profile_mean(const int32_t* budgets, float* profile, int n_queries, int64_t count, int n,
                                LaunchCtx& lc);
constexpr int kLookupSeqPerLaunch = 32;
cudaError_t launch_profile_budgets(const float* profile, const int* row_lo, const int* row_hi, const double* frac,
                                   const Dims& dm, int32_t* budgets, int32_t* offsets, LaunchCtx& lc);
// Curves of a proxy ranking: scores, importance [heads][n] -> curves [heads][P].
size_t curves_smem_bytes(int n, int P);
cudaError_t launch_build_curves(const Dims& dm, const float* scores, const float* importance, float* curves,
                                LaunchCtx& lc);
// KeyDiff proxy scores (key-only metric): scores [heads][n]; scratch of keydiff_scratch_bytes().
size_t keydiff_scratch_bytes(const Dims& dm);
cudaError_t launch_keydiff(const Dims& dm, const void* k, float* scores, float* scratch, int32_t* dev_status,
                           int spare_sms, LaunchCtx& lc);
// Value norms || v_j W_O^(g) ||_2 of the oracle importance on the tensor cores (bf16, d = 128): vnorm [heads][G][n].
bool value_norm_tc_supported(const Dims& dm);
cudaError_t launch_value_norm_tc(const Dims& dm, int d_model, const void* v, const void* w_o, float* vnorm,
                                 LaunchCtx& lc);
// Oracle importance of Sec. 4.1 from decode queries, the cache and the output projection.
size_t importance_workspace_bytes(const Dims& dm, int k_max);
cudaError_t launch_importance(const Dims& dm, int k_max, int d_model, const void* q_dec, const void* k, const void* v,
                              const void* k_dec, const void* w_o, bool normalize, float* importance, void* ws,
                              LaunchCtx& lc);
// Exact allocation (dynamic programme over the heads) at token resolution.
size_t exact_workspace_bytes(const Dims& dm, int64_t max_budget);
cudaError_t launch_exact_allocate(const Dims& dm, const float* curves, const int64_t* budgets_host, int32_t* budgets,
                                  int32_t* offsets, double* values, void* ws, LaunchCtx& lc);
cudaError_t launch_select(const Dims& dm, const float* scores, const int32_t* budgets, const int32_t* offsets,
                          int32_t* kept_idx, int64_t rows_cap, HeadRange hr, LaunchCtx& lc);
cudaError_t launch_gather(const Dims& dm, const int32_t* offsets, const int32_t* kept_idx, const void* k,
                          const void* v, void* k_out, void* v_out, int64_t rows_cap, HeadRange hr, LaunchCtx& lc);

}  // namespace lukv
