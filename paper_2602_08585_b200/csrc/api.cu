// C ABI of liblukv.so: argument validation, workspace carve-up and stage sequencing.
// Every step of the path runs in the kernels of this library; there is no host fallback.
#include <math.h>
#include <stdlib.h>

#include <mutex>

#include "common.cuh"

namespace lukv {

static thread_local int g_last_launches = 0;

static size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

Workspace carve_workspace(const Dims& dm, void* base) {
  Workspace ws;
  char* p = static_cast<char*>(base);
  size_t off = 0;
  auto take = [&](size_t bytes) {
    void* r = p ? p + off : nullptr;
    off += align256(bytes);
    return r;
  };
  const size_t heads = (size_t)dm.heads();
  ws.raw = static_cast<float*>(take(heads * dm.n * sizeof(float)));
  ws.pooled = static_cast<float*>(take(heads * dm.n * sizeof(float)));
  const size_t stats_simt = heads * score_chunks(dm) * dm.M * 2 * sizeof(float);
  size_t stats_bytes = score_tc_stats_bytes(dm);
  if (stats_simt > stats_bytes) stats_bytes = stats_simt;
  if (score_onepass_stats_bytes(dm) > stats_bytes) stats_bytes = score_onepass_stats_bytes(dm);
  if (keydiff_scratch_bytes(dm) > stats_bytes) stats_bytes = keydiff_scratch_bytes(dm);
  ws.stats = static_cast<float*>(take(stats_bytes));
  ws.lse = static_cast<float*>(take(heads * dm.M * sizeof(float)));
  ws.gains = static_cast<float*>(take((size_t)dm.N * (dm.P - 1) * sizeof(float)));
  ws.head_flags = static_cast<int*>(take(score_tc_flag_bytes(dm)));
  ws.bytes = off;
  return ws;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Per-sequence context lengths of a ragged call: w < T_q <= T, the curve grid must divide every length, the sinks
// must fit every sequence.  On success dm describes the longest sequence and carries the lengths.
static int attach_seq_lens(Dims* dm, const int32_t* ctx_lens) {
  if (!ctx_lens) return LUKV_ERR_INVALID_ARG;
  if (dm->S > kMaxRaggedSeqs || dm->keydiff) return LUKV_ERR_UNSUPPORTED;
  for (int q = 0; q < dm->S; ++q) {
    const int Tq = ctx_lens[q];
    if (Tq <= dm->w || Tq > dm->T || dm->n_sink > Tq - dm->w) return LUKV_ERR_INVALID_ARG;
    if (Tq % (dm->P - 1) != 0) return LUKV_ERR_UNSUPPORTED;
  }
  dm->seq_T = ctx_lens;
  return LUKV_OK;
}

// Validates the parameter block and fills Dims.
static int make_dims(const lukv_params_t* p, Dims* dm) {
  if (!p) return LUKV_ERR_INVALID_ARG;
  if ((p->flags & ~LUKV_FLAG_KEYDIFF) != 0) return LUKV_ERR_INVALID_ARG;
  if ((p->flags & LUKV_FLAG_KEYDIFF) && p->pool_kernel != 1) return LUKV_ERR_INVALID_ARG;
  if (p->batch < 1 || p->n_layers < 1 || p->n_kv_heads < 1 || p->gqa_group < 1 || p->ctx_len < 2 || p->window < 1 ||
      p->window >= p->ctx_len || p->pool_kernel < 1 || p->curve_points < 2)
    return LUKV_ERR_INVALID_ARG;
  if (!(p->softmax_scale >= 0.f) || isinf(p->softmax_scale)) return LUKV_ERR_INVALID_ARG;
  if (p->n_sink < 0 || p->n_sink > p->ctx_len - p->window || !(p->min_keep >= 0.f) || !(p->min_keep <= 1.f))
    return LUKV_ERR_INVALID_ARG;
  if (p->head_dim != 64 && p->head_dim != 128) return LUKV_ERR_UNSUPPORTED;
  if (p->dtype != LUKV_DTYPE_BF16 && p->dtype != LUKV_DTYPE_FP32) return LUKV_ERR_UNSUPPORTED;
  if ((p->pool_kernel & 1) == 0) return LUKV_ERR_UNSUPPORTED;
  if (p->curve_points > 4097) return LUKV_ERR_UNSUPPORTED;
  if (p->ctx_len % (p->curve_points - 1) != 0) return LUKV_ERR_UNSUPPORTED;
  if ((int64_t)p->gqa_group * p->window > 256) return LUKV_ERR_UNSUPPORTED;
  const int64_t N = (int64_t)p->n_layers * p->n_kv_heads;
  // the greedy kernel keeps three 32-bit indices per head in the shared memory of one CTA
  if (N > kGreedyMaxHeads) return LUKV_ERR_UNSUPPORTED;
  const int64_t heads = N * p->batch;
  // packed row indices, segment ids k*N+hid and grid sizes must fit 32 bits
  if (heads * p->ctx_len >= (int64_t)1 << 31 || N * (p->curve_points - 1) >= (int64_t)1 << 31 || heads > (1 << 24))
    return LUKV_ERR_UNSUPPORTED;
  dm->S = p->batch; dm->L = p->n_layers; dm->H = p->n_kv_heads; dm->G = p->gqa_group; dm->d = p->head_dim;
  dm->T = p->ctx_len; dm->w = p->window; dm->kp = p->pool_kernel; dm->dtype = p->dtype; dm->P = p->curve_points;
  dm->N = (int)N;
  dm->n = dm->T - dm->w;
  dm->M = dm->G * dm->w;
  dm->seg = dm->T / (dm->P - 1);
  dm->nseg = (dm->n + dm->seg - 1) / dm->seg;
  const float scale = p->softmax_scale > 0.f ? p->softmax_scale : (float)(1.0 / sqrt((double)dm->d));
  dm->scale_log2 = (float)((double)scale * 1.4426950408889634);
  dm->n_sink = p->n_sink;
  dm->min_keep = p->min_keep;
  dm->seq_T = nullptr;
  dm->keydiff = (p->flags & LUKV_FLAG_KEYDIFF) != 0;
  const double fl = ceil((double)p->min_keep * (double)dm->n);
  dm->floor_tok = fl < 0.0 ? 0 : (fl > (double)dm->n ? dm->n : (int)fl);
  return LUKV_OK;
}

static int check_budgets(const Dims& dm, const int64_t* budgets_in, int64_t* total_rows) {
  int64_t rows = 0;
  for (int q = 0; q < dm.S; ++q) {
    if (budgets_in[q] < (int64_t)dm.N * seq_floor_tokens(dm, q) || budgets_in[q] > (int64_t)dm.N * seq_rankable(dm, q))
      return LUKV_ERR_BUDGET;
    rows += budgets_in[q] + (int64_t)dm.N * dm.w;
  }
  *total_rows = rows;
  return LUKV_OK;
}

static int check_ws(const Dims& dm, void* ws, size_t ws_bytes, Workspace* out) {
  if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255u)) return LUKV_ERR_INVALID_ARG;
  *out = carve_workspace(dm, ws);
  if (ws_bytes < out->bytes) return LUKV_ERR_WORKSPACE_TOO_SMALL;
  return LUKV_OK;
}

// LUKV_FORCE_SIMT=1 routes every shape through the FP32-pipe scorer (for A/B checks).
static bool force_simt() {
  static const bool v = [] {
    const char* e = getenv("LUKV_FORCE_SIMT");
    return e && e[0] == '1';
  }();
  return v;
}

static HeadRange all_heads(const Dims& dm) { return HeadRange{0, (int)dm.heads()}; }

static cudaError_t run_score(const Dims& dm, const void* q, const void* k, const Workspace& ws, float* pooled_out,
                             int32_t* dev_status, LaunchCtx& lc) {
  if (dm.keydiff) return launch_keydiff(dm, k, pooled_out, ws.stats, dev_status, 0, lc);  // nothing to pool
  cudaError_t e = (score_tc_supported(dm) && !force_simt())
                      ? launch_score_tc(dm, q, k, ws, dev_status, all_heads(dm), true, 0, lc)
                      : launch_score_simt(dm, q, k, ws, lc);
  if (e != cudaSuccess) return e;
  return launch_pool(dm, ws.raw, pooled_out, all_heads(dm), lc);
}

// An auxiliary stream and the two events that tie it to the caller's stream, created on first
// use on a device and kept until the process exits (handles only, no device memory).
struct SideStream {
  cudaStream_t stream = nullptr;
  cudaEvent_t fork = nullptr, join = nullptr;
  bool ok = false;
  // held while a call records and waits on the two events: a second host thread that calls on the same
  // device must not re-record them between this call's record and the wait that belongs to it
  std::mutex use;
};
static SideStream* side_stream() {
  static SideStream table[64];
  static std::mutex mu;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lock(mu);
  SideStream& s = table[dev];
  if (!s.ok) {
    if (cudaStreamCreateWithFlags(&s.stream, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&s.fork, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&s.join, cudaEventDisableTiming) != cudaSuccess)
      return nullptr;
    s.ok = true;
  }
  return &s;
}

// The whole path.  Allocation depends only on the curves, scoring only on Q/K; selection needs
// both, the gather follows.  With `overlap` the two allocation kernels run on an auxiliary stream
// beside the scorer, which then leaves one SM to them (its CTAs fill theirs completely); the
// caller's stream waits for the budgets before selection, so stream order is preserved.
static int run_compress(const Dims& dm, const void* q_win, const void* k, const void* v, const float* curves,
                        const int64_t* budgets_in, void* k_out, void* v_out, int32_t* kept_idx, int32_t* budgets,
                        int32_t* offsets, int64_t rows_cap, int32_t* dev_status, const Workspace& w, LaunchCtx& lc,
                        bool overlap) {
  if (dev_status && cudaMemsetAsync(dev_status, 0, sizeof(int32_t), lc.st) != cudaSuccess) return LUKV_ERR_CUDA;
  const bool tc = score_tc_supported(dm) && !force_simt();
  // the persistent scorers (tensor-core, KeyDiff) leave one SM to the allocation kernels of the auxiliary stream;
  // the FP32-pipe scorer's ordinary grids simply share the SMs with them
  SideStream* side = overlap ? side_stream() : nullptr;
  int rc = LUKV_OK;
  if (side) {
    std::lock_guard<std::mutex> in_use(side->use);
    LaunchCtx ls;
    ls.st = side->stream;
    if (cudaEventRecord(side->fork, lc.st) != cudaSuccess || cudaStreamWaitEvent(ls.st, side->fork, 0) != cudaSuccess)
      return LUKV_ERR_CUDA;
    if (launch_allocate(dm, curves, budgets_in, w.gains, budgets, offsets, ls) != cudaSuccess) rc = LUKV_ERR_CUDA;
    if (cudaEventRecord(side->join, ls.st) != cudaSuccess) rc = LUKV_ERR_CUDA;
    lc.launches += ls.launches;
    if (rc == LUKV_OK && dm.keydiff) {
      if (launch_keydiff(dm, k, w.pooled, w.stats, dev_status, 1, lc) != cudaSuccess) rc = LUKV_ERR_CUDA;
    } else if (rc == LUKV_OK && tc) {
      if (launch_score_tc(dm, q_win, k, w, dev_status, all_heads(dm), true, 1, lc) != cudaSuccess ||
          launch_pool(dm, w.raw, w.pooled, all_heads(dm), lc) != cudaSuccess)
        rc = LUKV_ERR_CUDA;
    } else if (rc == LUKV_OK) {
      if (run_score(dm, q_win, k, w, w.pooled, dev_status, lc) != cudaSuccess) rc = LUKV_ERR_CUDA;
    }
    // join even after a failure: the caller's stream must not run ahead of work already enqueued
    if (cudaStreamWaitEvent(lc.st, side->join, 0) != cudaSuccess) rc = LUKV_ERR_CUDA;
    if (rc != LUKV_OK) return rc;
  } else {
    if (launch_allocate(dm, curves, budgets_in, w.gains, budgets, offsets, lc) != cudaSuccess) return LUKV_ERR_CUDA;
    if (run_score(dm, q_win, k, w, w.pooled, dev_status, lc) != cudaSuccess) return LUKV_ERR_CUDA;
  }
  if (launch_select(dm, w.pooled, budgets, offsets, kept_idx, rows_cap, all_heads(dm), lc) != cudaSuccess)
    return LUKV_ERR_CUDA;
  if (launch_gather(dm, offsets, kept_idx, k, v, k_out, v_out, rows_cap, all_heads(dm), lc) != cudaSuccess)
    return LUKV_ERR_CUDA;
  return LUKV_OK;
}

static int check_compress_args(const lukv_params_t* params, const void* q_win, const void* k, const void* v,
                               const float* curves, const int64_t* budgets_in, void* k_out, void* v_out,
                               int32_t* kept_idx, int32_t* budgets, int32_t* offsets, int64_t rows_cap, void* ws,
                               size_t ws_bytes, Dims* dm, Workspace* w, const int32_t* ctx_lens = nullptr,
                               bool ragged = false) {
  int rc = make_dims(params, dm);
  if (rc != LUKV_OK) return rc;
  if (ragged && (rc = attach_seq_lens(dm, ctx_lens)) != LUKV_OK) return rc;
  if (!k || !v || !curves || !budgets_in || !k_out || !v_out || !kept_idx || !budgets || !offsets ||
      !aligned16(k) || !aligned16(v) || !aligned16(k_out) || !aligned16(v_out))
    return LUKV_ERR_INVALID_ARG;
  if (!dm->keydiff && (!q_win || !aligned16(q_win))) return LUKV_ERR_INVALID_ARG;
  int64_t rows;
  if ((rc = check_budgets(*dm, budgets_in, &rows)) != LUKV_OK) return rc;
  if (rows >= (int64_t)1 << 31) return LUKV_ERR_UNSUPPORTED;
  if (rows_cap < rows) return LUKV_ERR_OUTPUT_TOO_SMALL;
  return check_ws(*dm, ws, ws_bytes, w);
}

}  // namespace lukv

using namespace lukv;

extern "C" {

int lukv_workspace_bytes(const lukv_params_t* params, size_t* bytes) {
  Dims dm;
  if (!bytes) return LUKV_ERR_INVALID_ARG;
  const int rc = make_dims(params, &dm);
  if (rc != LUKV_OK) return rc;
  *bytes = carve_workspace(dm, nullptr).bytes;
  return LUKV_OK;
}

int lukv_score(const lukv_params_t* params, const void* q_win, const void* k, float* scores, void* ws, size_t ws_bytes,
               void* stream) {
  Dims dm;
  int rc = make_dims(params, &dm);
  if (rc != LUKV_OK) return rc;
  if (!k || !scores || !aligned16(k) || (!dm.keydiff && (!q_win || !aligned16(q_win)))) return LUKV_ERR_INVALID_ARG;
  Workspace w;
  if ((rc = check_ws(dm, ws, ws_bytes, &w)) != LUKV_OK) return rc;
  LaunchCtx lc;
  lc.st = (cudaStream_t)stream;
  if (run_score(dm, q_win, k, w, scores, nullptr, lc) != cudaSuccess) return LUKV_ERR_CUDA;
  g_last_launches = lc.launches;
  return LUKV_OK;
}

int lukv_score_keydiff(const lukv_params_t* params, const void* k, float* scores, int32_t* dev_status, void* ws,
                       size_t ws_bytes, void* stream) {
  Dims dm;
  int rc = make_dims(params, &dm);
  if (rc != LUKV_OK) return rc;
  if (!k || !scores || !aligned16(k)) return LUKV_ERR_INVALID_ARG;
  Workspace w;
  if ((rc = check_ws(dm, ws, ws_bytes, &w)) != LUKV_OK) return rc;
  LaunchCtx lc;
  lc.st = (cudaStream_t)stream;
  if (dev_status && cudaMemsetAsync(dev_status, 0, sizeof(int32_t), lc.st) != cudaSuccess) return LUKV_ERR_CUDA;
  if (launch_keydiff(dm, k, scores, w.stats, dev_status, 0, lc) != cudaSuccess) return LUKV_ERR_CUDA;
  g_last_launches = lc.launches;
  return LUKV_OK;
}

int lukv_score_ragged(const lukv_params_t* params, const int32_t* ctx_lens, const void* q_win, const void* k,
                      float* scores, void* ws, size_t ws_bytes, void* stream) {
  Dims dm;
  int rc = make_dims(params, &dm);
  if (rc != LUKV_OK) return rc;
  if ((rc = attach_seq_lens(&dm, ctx_lens)) != LUKV_OK) return rc;
  if (!k || !scores || !aligned16(k) || (!dm.keydiff && (!q_win || !aligned16(q_win)))) return LUKV_ERR_INVALID_ARG;
  Workspace w;
  if ((rc = check_ws(dm, ws, ws_bytes, &w)) != LUKV_OK) return rc;
  LaunchCtx lc;
  lc.st = (cudaStream_t)stream;
  if (run_score(dm, q_win, k, w, scores, nullptr, lc) != cudaSuccess) return LUKV_ERR_CUDA;
  g_last_launches = lc.launches;
  return LUKV_OK;
}

int lukv_allocate(const lukv_params_t* params, const float* curves, const int64_t* budgets_in, int32_t* budgets,
                  int32_t* offsets, void* ws, size_t ws_bytes, void* stream) {
  Dims dm;
  int rc = make_dims(params, &dm);
  if (rc != LUKV_OK) return rc;
  if (!curves || !budgets_in || !budgets || !offsets) return LUKV_ERR_INVALID_ARG;
  int64_t rows;
  if ((rc = check_budgets(dm, budgets_in, &rows)) != LUKV_OK) return rc;
  if (rows >= (int64_t)1 << 31) return LUKV_ERR_UNSUPPORTED;
  Workspace w;
  if ((rc = check_ws(dm, ws, ws_bytes, &w)) != LUKV_OK) return rc;
  LaunchCtx lc;
  lc.st = (cudaStream_t)stream;
  if (launch_allocate(dm, curves, budgets_in, w.gains, budgets, offsets, lc) != cudaSuccess) return LUKV_ERR_CUDA;
  g_last_launches = lc.launches;
  return LUKV_OK;
}

static int select_gather_impl(const lukv_params_t* params, const int32_t* ctx_lens, bool ragged, const float* scores,
                              const int32_t* budgets, const int32_t* offsets, const void* k, const void* v, void* k_out,
                              void* v_out, int32_t* kept_idx, int64_t rows_cap, void* ws, size_t ws_bytes,
                              void* stream) {
  Dims dm;
  int rc = make_dims(params, &dm);
  if (rc != LUKV_OK) return rc;
  if (ragged && (rc = attach_seq_lens(&dm, ctx_lens)) != LUKV_OK) return rc;
  if (!scores || !budgets || !offsets || !k || !v || !k_out || !v_out || !kept_idx || rows_cap < 0 || !aligned16(k) ||
      !aligned16(v) || !aligned16(k_out) || !aligned16(v_out))
    return LUKV_ERR_INVALID_ARG;
  Workspace w;
  if ((rc = check_ws(dm, ws, ws_bytes, &w)) != LUKV_OK) return rc;
  LaunchCtx lc;
  lc.st = (cudaStream_t)stream;
  if (launch_select(dm, scores, budgets, offsets, kept_idx, rows_cap, all_heads(dm), lc) != cudaSuccess)
    return LUKV_ERR_CUDA;
  if (launch_gather(dm, offsets, kept_idx, k, v, k_out, v_out, rows_cap, all_heads(dm), lc) != cudaSuccess)
    return LUKV_ERR_CUDA;
  g_last_launches = lc.launches;
  return LUKV_OK;
}

int lukv_select_gather(const lukv_params_t* params, const float* scores, const int32_t* budgets, const int32_t* offsets,
                       const void* k, const void* v, void* k_out, void* v_out, int32_t* kept_idx, int64_t rows_cap,
                       void* ws, size_t ws_bytes, void* stream) {
  return select_gather_impl(params, nullptr, false, scores, budgets, offsets, k, v, k_out, v_out, kept_idx, rows_cap, ws,
                            ws_bytes, stream);
}

int lukv_select_gather_ragged(const lukv_params_t* params, const int32_t* ctx_lens, const float* scores,
                              const int32_t* budgets, const int32_t* offsets, const void* k, const void* v, void* k_out,
                              void* v_out, int32_t* kept_idx, int64_t rows_cap, void* ws, size_t ws_bytes,
                              void* stream) {
  return select_gather_impl(params, ctx_lens, true, scores, budgets, offsets, k, v, k_out, v_out, kept_idx, rows_cap, ws,
                            ws_bytes, stream);
}

int lukv_compress(const lukv_params_t* params, const void* q_win, const void* k, const void* v, const float* curves,
                  const int64_t* budgets_in, void* k_out, void* v_out, int32_t* kept_idx, int32_t* budgets,
                  int32_t* offsets, int64_t rows_cap, int32_t* dev_status, void* ws, size_t ws_bytes, void* stream) {
  Dims dm;
  Workspace w;
  int rc = check_compress_args(params, q_win, k, v, curves, budgets_in, k_out, v_out, kept_idx, budgets, offsets,
                               rows_cap, ws, ws_bytes, &dm, &w);
  if (rc != LUKV_OK) return rc;
  LaunchCtx lc;
  lc.st = (cudaStream_t)stream;
  rc = run_compress(dm, q_win, k, v, curves, budgets_in, k_out, v_out, kept_idx, budgets, offsets, rows_cap,
                    dev_status, w, lc, true);
  if (rc == LUKV_OK) g_last_launches = lc.launches;
  return rc;
}

int lukv_compress_ragged(const lukv_params_t* params, const int32_t* ctx_lens, const void* q_win, const void* k,
                         const void* v, const float* curves, const int64_t* budgets_in, void* k_out, void* v_out,
                         int32_t* kept_idx, int32_t* budgets, int32_t* offsets, int64_t rows_cap, int32_t* dev_status,
                         void* ws, size_t ws_bytes, void* stream) {
  Dims dm;
  Workspace w;
  int rc = check_compress_args(params, q_win, k, v, curves, budgets_in, k_out, v_out, kept_idx, budgets, offsets,
                               rows_cap, ws, ws_bytes, &dm, &w, ctx_lens, true);
  if (rc != LUKV_OK) return rc;
  LaunchCtx lc;
  lc.st = (cudaStream_t)stream;
  rc = run_compress(dm, q_win, k, v, curves, budgets_in, k_out, v_out, kept_idx, budgets, offsets, rows_cap,
                    dev_status, w, lc, true);
  if (rc == LUKV_OK) g_last_launches = lc.launches;
  return rc;
}

int lukv_compress_profile(const lukv_params_t* params, const void* q_win, const void* k, const void* v,
                          const float* curves, const int64_t* budgets_in, void* k_out, void* v_out,
                          int32_t* kept_idx, int32_t* budgets, int32_t* offsets, int64_t rows_cap,
                          int32_t* dev_status, void* ws, size_t ws_bytes, void* stream, lukv_kernel_time_t* times,
                          int max_times, int* n_times) {
  Dims dm;
  Workspace w;
  if (!times || !n_times || max_times < 1 || max_times > 64) return LUKV_ERR_INVALID_ARG;
  int rc = check_compress_args(params, q_win, k, v, curves, budgets_in, k_out, v_out, kept_idx, budgets, offsets,
                               rows_cap, ws, ws_bytes, &dm, &w);
  if (rc != LUKV_OK) return rc;
  cudaEvent_t ev[65];
  const char* names[64];
  for (int i = 0; i <= max_times; ++i)
    if (cudaEventCreate(&ev[i]) != cudaSuccess) {
      while (--i >= 0) cudaEventDestroy(ev[i]);
      return LUKV_ERR_CUDA;
    }
  LaunchCtx lc;
  lc.st = (cudaStream_t)stream;
  lc.events = ev;
  lc.names = names;
  lc.max_events = max_times;
  cudaEventRecord(ev[0], lc.st);
  rc = run_compress(dm, q_win, k, v, curves, budgets_in, k_out, v_out, kept_idx, budgets, offsets, rows_cap,
                    dev_status, w, lc, false);
  if (rc == LUKV_OK && cudaStreamSynchronize(lc.st) != cudaSuccess) rc = LUKV_ERR_CUDA;
  const int cnt = lc.launches < max_times ? lc.launches : max_times;
  if (rc == LUKV_OK) {
    for (int i = 0; i < cnt; ++i) {
      times[i].name = names[i];
      if (cudaEventElapsedTime(&times[i].ms, ev[i], ev[i + 1]) != cudaSuccess) rc = LUKV_ERR_CUDA;
    }
    *n_times = cnt;
    g_last_launches = lc.launches;
  }
  for (int i = 0; i <= max_times; ++i) cudaEventDestroy(ev[i]);
  return rc;
}

// ---- allocation without a caller-provided workspace ---------------------------------------
// Scratch of lukv_allocate_static: the hull gains [N][P-1].  The array lives in every GPU
// context that loads this library, from load until exit.
#define LUKV_STATIC_GAINS_MAX (256 * 1024)
static __device__ __align__(256) float g_static_gains[LUKV_STATIC_GAINS_MAX];

// In host code `g_static_gains` is only a handle for the runtime, not a device address; the
// address on the current device is looked up once per device and cached here.
static float* g_static_gains_ptr[64] = {nullptr};
static std::mutex g_static_gains_mutex;

static int static_gains_address(float** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return LUKV_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_static_gains_mutex);
  if (!g_static_gains_ptr[dev]) {
    float* ptr = nullptr;
    if (cudaGetSymbolAddress((void**)&ptr, g_static_gains) != cudaSuccess || !ptr) return LUKV_ERR_CUDA;
    g_static_gains_ptr[dev] = ptr;
  }
  *out = g_static_gains_ptr[dev];
  return LUKV_OK;
}

int lukv_allocate_static(const lukv_params_t* params, const float* curves, const int64_t* budgets_in,
                         int32_t* budgets, int32_t* offsets, void* stream) {
  Dims dm;
  int rc = make_dims(params, &dm);
  if (rc != LUKV_OK) return rc;
  if (!curves || !budgets_in || !budgets || !offsets) return LUKV_ERR_INVALID_ARG;
  if ((int64_t)dm.N * (dm.P - 1) > LUKV_STATIC_GAINS_MAX) return LUKV_ERR_WORKSPACE_TOO_SMALL;
  int64_t rows;
  if ((rc = check_budgets(dm, budgets_in, &rows)) != LUKV_OK) return rc;
  if (rows >= (int64_t)1 << 31) return LUKV_ERR_UNSUPPORTED;
  float* gains = nullptr;
  if ((rc = static_gains_address(&gains)) != LUKV_OK) return rc;
  LaunchCtx lc;
  lc.st = (cudaStream_t)stream;
  // the hull kernel overwrites gains[0 .. N*(P-1)) before the greedy kernel reads them, so
  // nothing left by an earlier call is ever consumed
  if (launch_allocate(dm, curves, budgets_in, gains, budgets, offsets, lc) != cudaSuccess) return LUKV_ERR_CUDA;
  g_last_launches = lc.launches;
  return LUKV_OK;
}

// ---- offline profile and online lookup (Sec. 4.3) -----------------------------------------

namespace {
struct ProfileWs {
  float* gains;      // [Mq][N][P-1]
  int32_t* budgets;  // [Mq][R][N]
  int32_t* offsets;  // [Mq][R*N+1] (written by the greedy kernel, not used further)
  size_t bytes;
};
ProfileWs carve_profile_ws(const Dims& dm, int n_queries, void* base) {
  ProfileWs ws;
  char* p = static_cast<char*>(base);
  size_t off = 0;
  auto take = [&](size_t bytes) {
    void* r = p ? p + off : nullptr;
    off += align256(bytes);
    return r;
  };
  const size_t Mq = (size_t)n_queries, RN = (size_t)dm.S * dm.N;
  ws.gains = static_cast<float*>(take(Mq * dm.N * (dm.P - 1) * sizeof(float)));
  ws.budgets = static_cast<int32_t*>(take(Mq * RN * sizeof(int32_t)));
  ws.offsets = static_cast<int32_t*>(take(Mq * (RN + 1) * sizeof(int32_t)));
  ws.bytes = off;
  return ws;
}
// Dims of the calibration problem: the n_ratios grid points take the place of the sequences.
int make_profile_dims(const lukv_params_t* calib, int32_t n_queries, int32_t n_ratios, Dims* dm) {
  if (!calib || n_queries < 1 || n_ratios < 1 || calib->batch != 1) return LUKV_ERR_INVALID_ARG;
  lukv_params_t p = *calib;
  p.batch = n_ratios;
  const int rc = make_dims(&p, dm);
  if (rc != LUKV_OK) return rc;
  if ((int64_t)n_queries * dm->N * (int64_t)dm->P >= (int64_t)1 << 31 || n_queries > 65535) return LUKV_ERR_UNSUPPORTED;
  return LUKV_OK;
}
}  // namespace

int lukv_profile_workspace_bytes(const lukv_params_t* calib, int32_t n_queries, int32_t n_ratios, size_t* bytes) {
  Dims dm;
  if (!bytes) return LUKV_ERR_INVALID_ARG;
  const int rc = make_profile_dims(calib, n_queries, n_ratios, &dm);
  if (rc != LUKV_OK) return rc;
  *bytes = carve_profile_ws(dm, n_queries, nullptr).bytes;
  return LUKV_OK;
}

int lukv_profile_build(const lukv_params_t* calib, const float* curves, int32_t n_queries, const float* ratios,
                       int32_t n_ratios, float* profile, void* ws, size_t ws_bytes, void* stream) {
  Dims dm;
  int rc = make_profile_dims(calib, n_queries, n_ratios, &dm);
  if (rc != LUKV_OK) return rc;
  if (!curves || !ratios || !profile || !ws || (reinterpret_cast<uintptr_t>(ws) & 255u)) return LUKV_ERR_INVALID_ARG;
  const ProfileWs w = carve_profile_ws(dm, n_queries, ws);
  if (ws_bytes < w.bytes) return LUKV_ERR_WORKSPACE_TOO_SMALL;
  // global budget of every grid point: B(rho) = floor((1 - rho) * N * n)
  int64_t* B = static_cast<int64_t*>(malloc(sizeof(int64_t) * (size_t)n_ratios));
  if (!B) return LUKV_ERR_CUDA;
  for (int j = 0; j < n_ratios; ++j) {
    const double rho = (double)ratios[j];
    if (!(rho >= 0.0 && rho <= 1.0)) {
      free(B);
      return LUKV_ERR_BUDGET;
    }
    B[j] = (int64_t)floor((1.0 - rho) * (double)((int64_t)dm.N * dm.n));
    if (B[j] < (int64_t)dm.N * dm.floor_tok) B[j] = (int64_t)dm.N * dm.floor_tok;
  }
  LaunchCtx lc;
  lc.st = (cudaStream_t)stream;
  cudaError_t e = launch_hull(curves, w.gains, (int64_t)n_queries * dm.N, dm.P, lc);
  if (e == cudaSuccess) e = launch_greedy(dm, w.gains, B, w.budgets, w.offsets, n_queries, lc);
  free(B);  // the budgets travel by value in the launch arguments
  if (e == cudaSuccess) e = launch_profile_mean(w.budgets, profile, n_queries, (int64_t)dm.S * dm.N, dm.n, lc);
  if (e != cudaSuccess) return LUKV_ERR_CUDA;
  g_last_launches = lc.launches;
  return LUKV_OK;
}

static int profile_budgets_impl(const lukv_params_t* params, const int32_t* ctx_lens, bool ragged, const float* profile,
                                const float* ratios, int32_t n_ratios, const float* sigma, int32_t* budgets,
                                int32_t* offsets, void* stream) {
  Dims dm;
  int rc = make_dims(params, &dm);
  if (rc != LUKV_OK) return rc;
  if (ragged && (rc = attach_seq_lens(&dm, ctx_lens)) != LUKV_OK) return rc;
  if (!profile || !ratios || !sigma || !budgets || !offsets || n_ratios < 1) return LUKV_ERR_INVALID_ARG;
  for (int j = 0; j + 1 < n_ratios; ++j)
    if (!(ratios[j] < ratios[j + 1])) return LUKV_ERR_INVALID_ARG;
  const size_t S = (size_t)dm.S;
  int* rows = static_cast<int*>(malloc(S * (2 * sizeof(int) + sizeof(double))));
  if (!rows) return LUKV_ERR_CUDA;
  int* row_lo = rows;
  int* row_hi = rows + S;
  double* frac = reinterpret_cast<double*>(rows + 2 * S);
  for (int q = 0; q < dm.S; ++q) {
    const float sg = sigma[q];
    if (!(sg >= ratios[0] && sg <= ratios[n_ratios - 1])) {
      free(rows);
      return LUKV_ERR_BUDGET;
    }
    int j = 0;
    while (j + 1 < n_ratios && ratios[j + 1] <= sg) ++j;
    const int j1 = j + 1 < n_ratios ? j + 1 : j;
    row_lo[q] = j;
    row_hi[q] = j1;
    frac[q] = j1 == j ? 0.0 : ((double)sg - (double)ratios[j]) / ((double)ratios[j1] - (double)ratios[j]);
  }
  LaunchCtx lc;
  lc.st = (cudaStream_t)stream;
  const cudaError_t e =
      launch_profile_budgets(profile, row_lo, row_hi, frac, dm, budgets, offsets, lc);
  free(rows);
  if (e != cudaSuccess) return LUKV_ERR_CUDA;
  g_last_launches = lc.launches;
  return LUKV_OK;
}

int lukv_profile_budgets(const lukv_params_t* params, const float* profile, const float* ratios, int32_t n_ratios,
                         const float* sigma, int32_t* budgets, int32_t* offsets, void* stream) {
  return profile_budgets_impl(params, nullptr, false, profile, ratios, n_ratios, sigma, budgets, offsets, stream);
}

int lukv_profile_budgets_ragged(const lukv_params_t* params, const int32_t* ctx_lens, const float* profile,
                                const float* ratios, int32_t n_ratios, const float* sigma, int32_t* budgets,
                                int32_t* offsets, void* stream) {
  return profile_budgets_impl(params, ctx_lens, true, profile, ratios, n_ratios, sigma, budgets, offsets, stream);
}

int lukv_build_curves(const lukv_params_t* params, const float* scores, const float* importance, float* curves,
                      void* stream) {
  Dims dm;
  int rc = make_dims(params, &dm);
  if (rc != LUKV_OK) return rc;
  if (!scores || !importance || !curves) return LUKV_ERR_INVALID_ARG;
  if (curves_smem_bytes(dm.n, dm.P) > 200u * 1024u) return LUKV_ERR_UNSUPPORTED;
  LaunchCtx lc;
  lc.st = (cudaStream_t)stream;
  if (launch_build_curves(dm, scores, importance, curves, lc) != cudaSuccess) return LUKV_ERR_CUDA;
  g_last_launches = lc.launches;
  return LUKV_OK;
}

int lukv_importance_workspace_bytes(const lukv_params_t* params, int32_t k_max, size_t* bytes) {
  Dims dm;
  if (!bytes || k_max < 1) return LUKV_ERR_INVALID_ARG;
  const int rc = make_dims(params, &dm);
  if (rc != LUKV_OK) return rc;
  if ((int64_t)dm.heads() * dm.G * k_max >= (int64_t)1 << 31) return LUKV_ERR_UNSUPPORTED;
  *bytes = importance_workspace_bytes(dm, k_max);
  return LUKV_OK;
}

int lukv_oracle_importance(const lukv_params_t* params, int32_t k_max, int32_t d_model, const void* q_dec,
                           const void* k, const void* v, const void* k_dec, const void* w_o, int32_t normalize,
                           float* importance, void* ws, size_t ws_bytes, void* stream) {
  Dims dm;
  int rc = make_dims(params, &dm);
  if (rc != LUKV_OK) return rc;
  if (k_max < 1 || d_model < 1 || !q_dec || !k || !v || !w_o || !importance || !ws ||
      (reinterpret_cast<uintptr_t>(ws) & 255u) || !aligned16(q_dec) || !aligned16(k) || !aligned16(v) ||
      (k_dec && !aligned16(k_dec)))
    return LUKV_ERR_INVALID_ARG;
  // grid dimensions: (heads * G) in x, tiles of 64 positions or blocks of 16 steps in y
  if ((int64_t)dm.heads() * dm.G * k_max >= (int64_t)1 << 31 || (dm.n + 63) / 64 > 65535 || (k_max + 15) / 16 > 65535)
    return LUKV_ERR_UNSUPPORTED;
  if (ws_bytes < importance_workspace_bytes(dm, k_max)) return LUKV_ERR_WORKSPACE_TOO_SMALL;
  LaunchCtx lc;
  lc.st = (cudaStream_t)stream;
  if (launch_importance(dm, k_max, d_model, q_dec, k, v, k_dec, w_o, normalize != 0, importance, ws, lc) != cudaSuccess)
    return LUKV_ERR_CUDA;
  g_last_launches = lc.launches;
  return LUKV_OK;
}

// Token resolution, no minimum retention: what the exact solver covers.
static int make_exact_dims(const lukv_params_t* params, Dims* dm) {
  const int rc = make_dims(params, dm);
  if (rc != LUKV_OK) return rc;
  if (dm->seg != 1 || dm->floor_tok != 0 || dm->n > 65535) return LUKV_ERR_UNSUPPORTED;
  return LUKV_OK;
}

int lukv_exact_workspace_bytes(const lukv_params_t* params, int64_t max_budget, size_t* bytes) {
  Dims dm;
  if (!bytes) return LUKV_ERR_INVALID_ARG;
  const int rc = make_exact_dims(params, &dm);
  if (rc != LUKV_OK) return rc;
  if (max_budget < 0 || max_budget > (int64_t)dm.N * dm.n) return LUKV_ERR_BUDGET;
  *bytes = exact_workspace_bytes(dm, max_budget);
  return LUKV_OK;
}

int lukv_exact_allocate(const lukv_params_t* params, const float* curves, const int64_t* budgets_in, int32_t* budgets,
                        int32_t* offsets, double* values, void* ws, size_t ws_bytes, void* stream) {
  Dims dm;
  int rc = make_exact_dims(params, &dm);
  if (rc != LUKV_OK) return rc;
  if (!curves || !budgets_in || !budgets || !offsets || !values || !ws || (reinterpret_cast<uintptr_t>(ws) & 255u))
    return LUKV_ERR_INVALID_ARG;
  int64_t rows, bmax = 0;
  if ((rc = check_budgets(dm, budgets_in, &rows)) != LUKV_OK) return rc;
  if (rows >= (int64_t)1 << 31) return LUKV_ERR_UNSUPPORTED;
  for (int q = 0; q < dm.S; ++q) bmax = budgets_in[q] > bmax ? budgets_in[q] : bmax;
  if (ws_bytes < exact_workspace_bytes(dm, bmax)) return LUKV_ERR_WORKSPACE_TOO_SMALL;
  LaunchCtx lc;
  lc.st = (cudaStream_t)stream;
  if (launch_exact_allocate(dm, curves, budgets_in, budgets, offsets, values, ws, lc) != cudaSuccess) return LUKV_ERR_CUDA;
  g_last_launches = lc.launches;
  return LUKV_OK;
}

const char* lukv_strerror(int code) {
  switch (code) {
    case LUKV_OK: return "ok";
    case LUKV_ERR_INVALID_ARG: return "invalid argument (null or misaligned pointer, non-positive size, flags != 0)";
    case LUKV_ERR_UNSUPPORTED: return "unsupported configuration (head_dim, dtype, even pool kernel, curve grid, G*w > 256 or sizes beyond 32 bits)";
    case LUKV_ERR_BUDGET: return "budget outside [N*ceil(min_keep*(T-w)), N*(T-w)], or a compression ratio outside its range";
    case LUKV_ERR_WORKSPACE_TOO_SMALL: return "workspace smaller than lukv_workspace_bytes()";
    case LUKV_ERR_OUTPUT_TOO_SMALL: return "rows_cap smaller than sum(B_q) + S*N*w";
    case LUKV_ERR_CUDA: return "CUDA launch failed";
    case LUKV_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    default: return "unknown status";
  }
}

int lukv_last_launch_count(void) { return g_last_launches; }

}  // extern "C"
