/*
 * lukv.h -- C ABI of the LU-KV prefill-time KV-cache compression path for NVIDIA B200
 * (sm_100a).  Four stages, all executed by hand-written CUDA kernels inside liblukv.so:
 *
 *   score     proxy importance of every cached position, per KV head
 *   allocate  split a global token budget over the heads (hull relaxation + greedy)
 *   select    per-head top-b positions by score
 *   gather    compact the kept K/V rows (plus the always-kept observation window)
 *
 * Beside the four stages the library has the paper's profile mode (lukv_profile_build,
 * lukv_profile_budgets: Sec. 4.3), the curve builder that feeds it (lukv_build_curves), an
 * exact solver for cross-checks (lukv_exact_allocate) and a variant of the allocation that needs
 * no caller scratch (lukv_allocate_static).
 *
 * Problem statement implemented (paper Sec. 4.2 Eq. "combinatorial_optimization" and its
 * relaxed form, Sec. 4.3 "Online Execution"): given per-head utility-versus-budget
 * curves, a global budget and the prefill KV cache, produce integer per-head budgets b
 * with sum(b) = B exactly and, for every head, the retained set M^pi(b) of its top-b
 * positions under the proxy metric pi (SnapKV-style observation-window attention).
 *
 * Conventions
 *   - Every pointer is DEVICE memory unless marked HOST.  The caller owns every buffer;
 *     the library allocates no device memory, keeps no results between calls and never
 *     synchronises the stream.  All work is ordered on `stream` (a cudaStream_t passed as
 *     void*).
 *   - Tensors are contiguous, row-major, in the layouts written next to each argument.
 *   - Notation: S sequences, L layers, H KV heads per layer, N = L*H heads per sequence,
 *     G query heads per KV head, d head dim, T context length, w observation window,
 *     n = T-w rankable positions, kp max-pool width, P curve points per head,
 *     s = T/(P-1) tokens per curve segment.  Head index u = (q*L + l)*H + h; the head id
 *     inside a sequence is hid = l*H + h.
 *   - Return value: 0 (LUKV_OK) or a negative lukv_status.  Argument errors are detected
 *     on the host before anything is launched.  Inputs are assumed finite.
 */
#ifndef LUKV_H_
#define LUKV_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define LUKV_API __attribute__((visibility("default")))
#else
#define LUKV_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum lukv_status {
  LUKV_OK = 0,
  LUKV_ERR_INVALID_ARG = -1,         /* null pointer, non-positive size, unknown flag bits     */
  LUKV_ERR_UNSUPPORTED = -2,         /* d not in {64,128}, unknown dtype, even kp, (P-1) does  */
                                     /* not divide T, G*w > 256, P > 4097, N > 18944, sizes    */
                                     /* beyond int32                                           */
  LUKV_ERR_BUDGET = -3,              /* some B_q < 0 or B_q > N*n; a ratio outside its range   */
  LUKV_ERR_WORKSPACE_TOO_SMALL = -4, /* ws_bytes < lukv_workspace_bytes()                      */
  LUKV_ERR_OUTPUT_TOO_SMALL = -5,    /* rows_cap < sum_q B_q + S*N*w                           */
  LUKV_ERR_CUDA = -6,                /* a launch failed; cudaGetLastError() is left set        */
  LUKV_ERR_TIMEOUT = -7              /* written to *dev_status only: a bounded device wait ran */
                                     /* out; outputs of that call are unspecified              */
} lukv_status;

enum { LUKV_DTYPE_BF16 = 0, LUKV_DTYPE_FP32 = 1 };

/*
 * lukv_params_t.flags.  LUKV_FLAG_KEYDIFF: the proxy metric of stage (a) is KeyDiff (see lukv_score_keydiff)
 * instead of the observation-window attention scores, in lukv_score, lukv_compress and
 * lukv_compress_profile: q_win is ignored and may be NULL, gqa_group plays no role, pool_kernel must be 1 (the
 * metric is not pooled); App. E pairs it with window = 1.  The calls for sequences of different lengths return
 * LUKV_ERR_UNSUPPORTED with this flag.
 */
#define LUKV_FLAG_KEYDIFF 1

typedef struct lukv_params {
  int32_t batch;        /* S >= 1                                                             */
  int32_t n_layers;     /* L >= 1                                                             */
  int32_t n_kv_heads;   /* H >= 1, N = L*H <= 18944 (the greedy keeps 12 bytes of shared      */
                        /* memory per head of a sequence)                                     */
  int32_t gqa_group;    /* G >= 1, G*w <= 256                                                 */
  int32_t head_dim;     /* d in {64, 128}                                                     */
  int32_t ctx_len;      /* T                                                                  */
  int32_t window;       /* w, 1 <= w < T                                                      */
  int32_t pool_kernel;  /* kp, odd, >= 1                                                      */
  int32_t dtype;        /* LUKV_DTYPE_BF16 or LUKV_DTYPE_FP32: element type of Q, K and V     */
  int32_t curve_points; /* P, 2 <= P <= 4097, (P-1) divides T                                 */
  float softmax_scale;  /* 0 selects 1/sqrt(d) (Eq. 1)                                        */
  int32_t flags;        /* 0, or LUKV_FLAG_KEYDIFF; other bits must be 0                      */
  /* Deployment settings of App. E (implementation details); 0 switches either off.            */
  int32_t n_sink;       /* attention sinks: positions 0..n_sink-1 rank before all others in   */
                        /* the selection whatever their score, so they are kept whenever the  */
                        /* head's budget allows and count towards it; 0 <= n_sink <= n        */
                        /* (the paper uses 4)                                                 */
  float min_keep;       /* minimum retention per head, 0 <= min_keep <= 1 (the paper uses     */
                        /* 0.01): every head keeps at least f = ceil(min_keep * n) of its n   */
                        /* rankable tokens (fp64 product of the fp32 value).  Allocation      */
                        /* hands every head its first f tokens before the greedy spends       */
                        /* B_q - N*f (B_q < N*f is LUKV_ERR_BUDGET); the profile build        */
                        /* solves max(B(rho), N*f); the lookup raises budgets below f to f    */
} lukv_params_t;

/* Bytes of scratch that any of the calls below needs for these parameters (one size fits
 * all four).  The scratch must be 256-byte aligned.  Contents need no initialisation and
 * are undefined afterwards. */
LUKV_API int lukv_workspace_bytes(const lukv_params_t* params, size_t* bytes /* HOST, out */);

/*
 * Stage (a): proxy scoring.  Attention weights follow Eq. 1 (Sec. 3.1): softmax of
 * scale * <q, k>.  The proxy is the SnapKV observation-window score the paper adopts as
 * pi_1 (Sec. 5.1; window 32 / kernel 7 in its hyper-parameter table): for KV head u, the
 * queries are the last w positions of its G query heads; the query at position n+i sees
 * keys 0..n+i (causal); each row is soft-maxed over its visible keys; the probabilities
 * are summed over the w rows and the G query heads; the resulting vector over the n
 * non-window positions is max-pooled (width kp, stride 1, centred, clipped at the ends).
 *
 *   q_win  [S][L][H*G][w][d]  the queries of the last w positions (query head h*G+g
 *                             belongs to KV head h)
 *   k      [S][L][H][T][d]
 *   scores [S][N][n] fp32     out: pooled scores (>= 0)
 * This call has no device status word: should a bounded wait of the scorer run out (see dev_status of
 * lukv_compress; it needs the device to be taken away in mid-kernel), the scores are undefined and nothing
 * reports it.  lukv_compress and lukv_score_keydiff report it.
 */
LUKV_API int lukv_score(const lukv_params_t* params, const void* q_win, const void* k, float* scores, void* ws,
               size_t ws_bytes, void* stream);

/*
 * Stage (a) with the second proxy metric the paper evaluates, KeyDiff (pi_2 of Sec. 5.1; App. E uses a recent
 * window of 1 with it).  The paper only names the metric (as one that looks at the geometry of the key vectors);
 * the formula implemented is the one of the method's own publication: with u_j = k_j / max(||k_j||, eps) and the anchor
 * a = mean of u_j over all T cached keys of the head,
 *     scores[j] = - <k_j, a> / (max(||k_j||, eps) * max(||a||, eps)),   eps = 1e-8,
 * for the n = T-w rankable positions: keys far from the head's mean key direction score high and are kept first.
 * No queries, no pooling (pool_kernel must be valid but is unused).  The scores lie in [-1, 1]; they feed
 * lukv_select_gather and lukv_build_curves like the scores of lukv_score.
 *
 *   k          [S][L][H][T][d]
 *   scores     [S][N][n] fp32     out
 *   dev_status [1] int32, may be NULL: set to 0 by the call; LUKV_ERR_TIMEOUT if a bounded wait ran out (the
 *              kernel's CTAs wait for one another's partial sums of a head; it is launched cooperatively, so
 *              this only happens if the device is taken away).  The scores are then undefined.
 */
LUKV_API int lukv_score_keydiff(const lukv_params_t* params, const void* k, float* scores, int32_t* dev_status, void* ws,
                       size_t ws_bytes, void* stream);

/*
 * Stage (b): global head-level budget allocation (Sec. 4.2; App. A.2).
 * (b1) Hull relaxation: the P-1 increments of each head's utility curve are projected by
 *      pool-adjacent-violators onto a non-increasing sequence and clipped at 0
 *      (Eq. "marginal_gain"), in fp64, each gain rounded once to fp32.  Utility is
 *      U(b) = L(0) - L(b), so these are the paper's marginal decreases of the loss.
 * (b2) Greedy: curve point k is the utility of keeping the top k*s non-window tokens; all
 *      tokens of segment k share its gain, and the segment can hold
 *      cap = clamp(n - k*s, 0, s) tokens.  Segments are consumed in the order
 *      (gain descending, k ascending, hid ascending) until B_q tokens are spent, the last
 *      one partially -- the B_q largest marginal gains under the per-head prefix
 *      constraint.  sum_hid budgets[q][hid] == B_q exactly.
 *
 *   curves     [N][P] fp32          utility curves, shared by all sequences
 *   budgets_in [S] int64, HOST      selectable tokens B_q per sequence, 0 <= B_q <= N*n
 *                                   (window rows are kept on top of it)
 *   budgets    [S][N] int32         out
 *   offsets    [S*N+1] int32        out: exclusive scan of (budgets + w) over u; head u
 *                                   owns packed rows [offsets[u], offsets[u+1])
 */
LUKV_API int lukv_allocate(const lukv_params_t* params, const float* curves, const int64_t* budgets_in, int32_t* budgets,
                  int32_t* offsets, void* ws, size_t ws_bytes, void* stream);

/*
 * Stages (c)+(d): per-head top-b selection (Sec. 4.3 "Eviction": keep M^pi(b), the first b
 * positions when ranked by score descending; ties go to the lower position, the fixed
 * deterministic rule App. A.1 asks for) and compaction of the retained set (Sec. 3.2).
 * For head u with b = budgets[u] and o = offsets[u]:
 *   kept_idx[o .. o+b)      the selected positions, ascending
 *   kept_idx[o+b .. o+b+w)  the window positions n .. T-1
 *   k_out / v_out row r     = k / v row kept_idx[r] of head u, copied bit for bit
 *
 *   scores   [S][N][n] fp32   scores of the rankable positions (finite; any sign)
 *   budgets  [S][N] int32, offsets [S*N+1] int32   as produced by lukv_allocate; the
 *            caller guarantees 0 <= budgets <= n and offsets consistent with them
 *   k, v     [S][L][H][T][d]
 *   k_out, v_out [rows_cap][d], kept_idx [rows_cap] int32   out
 *   rows_cap rows available in the outputs; total rows = sum_q B_q + S*N*w is known on
 *            the host.  Rows at or beyond rows_cap are never written.
 */
LUKV_API int lukv_select_gather(const lukv_params_t* params, const float* scores, const int32_t* budgets,
                       const int32_t* offsets, const void* k, const void* v, void* k_out, void* v_out,
                       int32_t* kept_idx, int64_t rows_cap, void* ws, size_t ws_bytes, void* stream);

/*
 * The whole path in one call: score, allocate, select, gather (Sec. 4.2-4.3), with the
 * intermediate scores kept in the workspace.  Arguments as above.  Returns
 * LUKV_ERR_OUTPUT_TOO_SMALL when rows_cap < sum_q B_q + S*N*w.
 *   dev_status [1] int32, may be NULL: set to 0 by the call; a kernel that gives up on a
 *   bounded wait stores LUKV_ERR_TIMEOUT there (the tensor-core scorer's CTAs wait for one
 *   another; it is launched cooperatively, so this only happens if the device is taken away).
 * The allocation kernels run on an auxiliary stream beside the scorer; that stream and two
 * events are created on the first call on a device and kept until the process exits.  The
 * caller's stream waits for them inside the call, so everything the call enqueues is ordered
 * after earlier work on `stream` and before later work on it.  Host threads may call
 * concurrently on one device (each with its own workspace and outputs): the call holds a
 * per-device lock while it enqueues on the auxiliary stream, so such calls enqueue one after
 * the other.  The call only enqueues (kernels, memsets, the event pair), so it may be captured into a CUDA
 * graph once the auxiliary stream exists (after one plain call on the device).
 */
LUKV_API int lukv_compress(const lukv_params_t* params, const void* q_win, const void* k, const void* v,
                  const float* curves, const int64_t* budgets_in, void* k_out, void* v_out, int32_t* kept_idx,
                  int32_t* budgets, int32_t* offsets, int64_t rows_cap, int32_t* dev_status, void* ws,
                  size_t ws_bytes, void* stream);

/*
 * The same for a batch whose sequences have different context lengths, in one set of launches (App. E runs the
 * method on whatever context a request brings; Sec. 5.3: budgets are known before prefill, so nothing forces
 * sequences of one length into a call).  Sequence q has ctx_lens[q] cached positions, w < ctx_lens[q] <= T, of
 * which the last w are its observation window and the first n_q = ctx_lens[q] - w are rankable.
 *   - params->ctx_len = T is the ROW STRIDE of the cache: k, v are [S][L][H][T][d] with sequence q using the
 *     first ctx_lens[q] rows of each of its heads (the rest is padding and is never read as data);
 *     scores (lukv_score_ragged) are [S][N][T-w] with the first n_q entries of a row written.
 *   - The curve grid is per sequence: segment size ctx_lens[q]/(P-1), so (P-1) must divide every length
 *     (LUKV_ERR_UNSUPPORTED otherwise); 0 <= B_q <= N*n_q; min_keep gives ceil(min_keep*n_q) per head of q.
 *   - Outputs as in lukv_compress: head u of sequence q keeps budgets[u] positions of [0, n_q) and its window rows
 *     n_q .. ctx_lens[q]-1; rows = sum_q B_q + S*N*w.
 * ctx_lens [S] int32, HOST, read before the call returns; S <= 64.  The result equals what S single-sequence
 * calls (params with batch 1 and ctx_len = ctx_lens[q]) would produce, concatenated.
 */
LUKV_API int lukv_score_ragged(const lukv_params_t* params, const int32_t* ctx_lens, const void* q_win, const void* k,
                               float* scores, void* ws, size_t ws_bytes, void* stream);
LUKV_API int lukv_compress_ragged(const lukv_params_t* params, const int32_t* ctx_lens, const void* q_win,
                                  const void* k, const void* v, const float* curves, const int64_t* budgets_in,
                                  void* k_out, void* v_out, int32_t* kept_idx, int32_t* budgets, int32_t* offsets,
                                  int64_t rows_cap, int32_t* dev_status, void* ws, size_t ws_bytes, void* stream);
/*
 * Stages (c) and (d) for such a batch, for callers that bring their own budgets -- with lukv_profile_budgets_ragged
 * and lukv_score_ragged this is the paper's deployment mode (Sec. 4.3 "Online Execution") on sequences of different
 * lengths.  Arguments as lukv_select_gather; scores [S][N][T-w] with the first n_q entries of a row read;
 * 0 <= budgets[u] <= n_q; head u of sequence q keeps its window rows n_q .. ctx_lens[q]-1.
 */
LUKV_API int lukv_select_gather_ragged(const lukv_params_t* params, const int32_t* ctx_lens, const float* scores,
                                       const int32_t* budgets, const int32_t* offsets, const void* k, const void* v,
                                       void* k_out, void* v_out, int32_t* kept_idx, int64_t rows_cap, void* ws,
                                       size_t ws_bytes, void* stream);

/*
 * Profiling variant of lukv_compress (the paper has no counterpart): same arguments and
 * results, but a CUDA event is recorded after every kernel and the call SYNCHRONISES the
 * stream before returning the per-kernel device times.  Not for production use.
 *   times [max_times] HOST, out: kernel name (static string) and milliseconds, in launch
 *   order; n_times HOST, out: entries written.  1 <= max_times <= 64.
 */
typedef struct lukv_kernel_time {
  const char* name;
  float ms;
} lukv_kernel_time_t;
LUKV_API int lukv_compress_profile(const lukv_params_t* params, const void* q_win, const void* k, const void* v,
                                   const float* curves, const int64_t* budgets_in, void* k_out, void* v_out,
                                   int32_t* kept_idx, int32_t* budgets, int32_t* offsets, int64_t rows_cap,
                                   int32_t* dev_status, void* ws, size_t ws_bytes, void* stream,
                                   lukv_kernel_time_t* times, int max_times, int* n_times);

/*
 * lukv_allocate for callers that cannot hand over device scratch (the paper has no
 * counterpart; this is a packaging variant of stage (b)).  Some hosts of this library may
 * not call cudaMalloc at the point where budgets are needed -- a serving process whose
 * device memory is fully owned by its own pool allocator, or code running inside a region
 * where allocation is forbidden -- and so have no workspace to pass.  This entry point takes
 * none: the hull gains go to a fixed array of LUKV_STATIC_GAINS_MAX = 262144 floats (1 MiB)
 * that is part of the library image and is resident on every GPU that loads the library
 * until the process exits.  It calls no allocating routine.
 *
 *   - Limit: N*(P-1) <= 262144 (e.g. 256 heads x 1025 points); larger problems return
 *     LUKV_ERR_WORKSPACE_TOO_SMALL and launch nothing.
 *   - The first call on each device looks up the array's device address (a one-time runtime
 *     query, cached per device); make that first call before any stream capture begins.
 *   - All calls on a device share the one array.  It keeps the previous call's contents,
 *     which is harmless: every call rewrites the gains it uses before reading them.  Calls
 *     whose kernels can overlap on the GPU (different streams, or threads) race on it and
 *     must be serialised by the caller.
 *   - Arguments, results and error codes otherwise as lukv_allocate (no ws, ws_bytes).
 */
LUKV_API int lukv_allocate_static(const lukv_params_t* params, const float* curves, const int64_t* budgets_in,
                                  int32_t* budgets, int32_t* offsets, void* stream);

/*
 * Offline profile (Sec. 4.3 "Offline Optimal Budget Estimation", Eq. "calibration_avg").
 * Input: the per-head utility curves of n_queries calibration queries on one calibration
 * context (the paper uses about 4,000 tokens and 30 queries) and a grid of n_ratios global
 * compression ratios.  For every query and every grid ratio rho the relaxed allocation
 * problem of stage (b) is solved for the global budget B(rho) = floor((1-rho)*N*n), n = T-w
 * being the rankable positions of the calibration context; the query's optimal local ratio
 * of head hid is r* = 1 - b_hid/n; the profile entry is the mean of r* over the queries
 * (fp64, rounded once to fp32).  Token resolution is P = T+1 (s = 1).
 *
 *   calib     the calibration shape: n_layers, n_kv_heads, ctx_len, window, curve_points as
 *             in stage (b); batch must be 1; the other fields must be valid but are unused
 *   curves    [n_queries][N][P] fp32
 *   ratios    [n_ratios] fp32, HOST   each in [0,1] (else LUKV_ERR_BUDGET); read before
 *             the call returns
 *   profile   [n_ratios][N] fp32      out; 0 = keep everything, 1 = evict everything
 *   ws        lukv_profile_workspace_bytes() bytes, 256-byte aligned
 * Limits: N*n_ratios*T < 2^31, n_queries*N*P < 2^31, n_queries <= 65535.
 */
LUKV_API int lukv_profile_workspace_bytes(const lukv_params_t* calib, int32_t n_queries, int32_t n_ratios,
                                          size_t* bytes /* HOST, out */);
LUKV_API int lukv_profile_build(const lukv_params_t* calib, const float* curves, int32_t n_queries,
                                const float* ratios, int32_t n_ratios, float* profile, void* ws, size_t ws_bytes,
                                void* stream);

/*
 * Online lookup and budgeting (Sec. 4.3 "Online Execution", steps 1 and 2), the paper's
 * deployment front end in place of lukv_allocate: sequence q with target global compression
 * ratio sigma[q] takes the profile row at sigma[q] -- linearly interpolated between the two
 * neighbouring grid rows when sigma[q] is not a grid point (the paper leaves that case
 * open) -- and every head gets b = floor((1-r)*n), n = T-w of the NEW context described by
 * `params`, clamped to [0,n]; all in fp64.  The budgets of a sequence add up to at most
 * (1-sigma)*N*n and miss it by less than one token per head (plus the fp32 rounding of the
 * profile); unlike lukv_allocate the sum is not exact.  Step 3 (eviction) is
 * lukv_score followed by lukv_select_gather with these budgets and offsets.
 *
 *   profile   [n_ratios][N] fp32       as produced by lukv_profile_build (same N)
 *   ratios    [n_ratios] fp32, HOST    strictly ascending (else LUKV_ERR_INVALID_ARG)
 *   sigma     [S] fp32, HOST           ratios[0] <= sigma[q] <= ratios[n_ratios-1]
 *                                      (else LUKV_ERR_BUDGET); both read before return
 *   budgets   [S][N] int32             out
 *   offsets   [S*N+1] int32            out: exclusive scan of (budgets + w); the total row
 *                                      count offsets[S*N] is at most S*N*T
 */
LUKV_API int lukv_profile_budgets(const lukv_params_t* params, const float* profile, const float* ratios,
                                  int32_t n_ratios, const float* sigma, int32_t* budgets, int32_t* offsets,
                                  void* stream);
/*
 * The same for sequences of different context lengths (see lukv_compress_ragged for ctx_lens): head h of sequence
 * q gets b = floor((1-r)*n_q), n_q = ctx_lens[q] - w, raised to ceil(min_keep*n_q); the result equals one
 * single-sequence call per sequence, concatenated (offsets running over all sequences).
 */
LUKV_API int lukv_profile_budgets_ragged(const lukv_params_t* params, const int32_t* ctx_lens, const float* profile,
                                         const float* ratios, int32_t n_ratios, const float* sigma,
                                         int32_t* budgets, int32_t* offsets, void* stream);

/*
 * Utility-versus-budget curves of the proxy metric (Sec. 3.2: M^pi(k) is the set of the first k
 * positions in the ranking of pi; Eq. "head_loss_def": the eviction loss of a retained set is the
 * oracle importance mass outside it).  For every head, U(k) = L(empty) - L(M^pi(k)) is the
 * importance mass of its k highest-ranked positions; the curve handed to stage (b) and to the
 * profile build is U sampled every s = T/(P-1) tokens: curves[u][k] = U(min(k*s, n)).
 * The ranking is the selection's (sinks first, score descending, lower position first among
 * equals).  Sums are fp64 in ranking order, each point rounded once to fp32.  With S calibration
 * queries as the batch, the output is the [n_queries][N][P] input of lukv_profile_build.
 * The oracle importance (Eq. "oracle_importance") is an input here; lukv_oracle_importance computes it from
 * decode queries, the cache and the output projection.
 *
 *   scores      [S][N][n] fp32   proxy scores of the rankable positions (lukv_score)
 *   importance  [S][N][n] fp32   oracle importance of the same positions
 *   curves      [S][N][P] fp32   out; curves[..][0] = 0, non-decreasing for importance >= 0
 * Every position is ranked by counting the positions ahead of it (quadratic in n, no scratch
 * memory), which suits calibration contexts of a few thousand tokens; n beyond about 24,000
 * (8*n + 8*P bytes of shared memory above 200 KiB) returns LUKV_ERR_UNSUPPORTED.
 */
LUKV_API int lukv_build_curves(const lukv_params_t* params, const float* scores, const float* importance,
                               float* curves, void* stream);

/*
 * Oracle importance (Sec. 4.1, Eq. "oracle_importance"): the largest contribution a cached position makes to
 * the head output over K_max future decode steps,
 *     I_j = max_{k = 1..K_max}  A_{k,j} * || v_j W_O ||_2 ,
 * A_{k,j} being the attention weight (Eq. 1) of the query of decode step k on cached position j and W_O the
 * head's slice of the output projection; App. E names the L2 norm and an intra-layer normalisation.  An offline
 * analysis tool: its output, with the proxy scores of the same context, is the input of lukv_build_curves.
 * Where the paper leaves a choice:
 *   - the softmax of step k runs over the T cached positions and, if k_dec is given, over the keys of decode
 *     steps 1..k as well (the step's own key included); k_dec = NULL restricts it to the cached positions;
 *   - a KV head is read by G query heads, each with its own slice of W_O: their contributions are added before
 *     the maximum over the steps, I_j = max_k sum_g A_{g,k,j} * || v_j W_O^(g) ||_2 (G = 1: the formula above);
 *   - normalize != 0: every layer's values are divided by their sum over the layer's H heads and n rankable
 *     positions (fp64 total), so each layer of each sequence carries unit mass; 0 leaves them as they are.
 * Window positions are always kept and get no value: the output covers the n = T-w rankable positions.
 *
 *   q_dec       [S][L][H*G][k_max][d]   queries of the k_max decode steps (query head h*G+g reads KV head h)
 *   k, v        [S][L][H][T][d]         the prefill cache
 *   k_dec       [S][L][H][k_max][d]     keys of the decode steps, or NULL
 *   w_o         [L][H*G][d][d_model]    output projection, one [d][d_model] slice per query head, in the
 *                                       element type of the cache
 *   importance  [S][N][n] fp32          out
 *   ws          lukv_importance_workspace_bytes() bytes, 256-byte aligned (value norms and row log-sum-exps)
 * fp32 arithmetic on the inputs as given; params->pool_kernel and curve_points must be valid but are unused.
 */
LUKV_API int lukv_importance_workspace_bytes(const lukv_params_t* params, int32_t k_max, size_t* bytes /* HOST, out */);
LUKV_API int lukv_oracle_importance(const lukv_params_t* params, int32_t k_max, int32_t d_model, const void* q_dec,
                                    const void* k, const void* v, const void* k_dec, const void* w_o,
                                    int32_t normalize, float* importance, void* ws, size_t ws_bytes, void* stream);

/*
 * Exact allocation (Sec. 4.2, Eq. "combinatorial_optimization": maximise the summed utility over
 * integer budgets with sum b = B on the curves as given, no relaxation; the paper names the exact
 * solver as the comparison point of its relaxation).  A tool for cross-checks, not part of the
 * hot path: the multiple-choice-knapsack recursion over the heads, N*B*n/2 additions in fp32, one
 * launch per head.  Token-resolution curves only (P = T+1, so s = 1), n <= 65535, min_keep = 0;
 * anything else is LUKV_ERR_UNSUPPORTED.
 *
 *   curves      [N][P] fp32          as in lukv_allocate (need not be monotone or concave)
 *   budgets_in  [S] int64, HOST      0 <= B_q <= N*n
 *   budgets     [S][N] int32         out: one optimal solution (ties: the smallest budget for the
 *                                    later head); sum_hid budgets[q][hid] == B_q
 *   offsets     [S*N+1] int32        out, as in lukv_allocate
 *   values      [S] fp64             out: the optimum (accumulated in fp32)
 *   ws          lukv_exact_workspace_bytes(params, max_q B_q) bytes, 256-byte aligned:
 *               two fp32 rows of B+1 values and the 16-bit argmax of every (head, budget)
 */
LUKV_API int lukv_exact_workspace_bytes(const lukv_params_t* params, int64_t max_budget, size_t* bytes /* HOST, out */);
LUKV_API int lukv_exact_allocate(const lukv_params_t* params, const float* curves, const int64_t* budgets_in,
                                 int32_t* budgets, int32_t* offsets, double* values, void* ws, size_t ws_bytes,
                                 void* stream);

/* Static description of a status code. */
LUKV_API const char* lukv_strerror(int code);

/* Number of kernels the last successful call on this thread enqueued (for accounting). */
LUKV_API int lukv_last_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* LUKV_H_ */
