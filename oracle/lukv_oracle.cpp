// LU-KV prefill compression path -- CPU ORACLE (test infrastructure, not product code).
//
// A plain, slow, single-threaded restatement of what the path computes, in double
// precision, written from the paper's definitions and used only to check the CUDA
// library: the tests, the smoke check and the benchmark's CPU-baseline leg call it.
// It shares no code, header, table or helper with the CUDA path and must never be
// reached from the product path.
//
// Stages (each function cites the passage it follows):
//   score    : SnapKV-style observation-window proxy. Attention weights are the
//              scaled-dot-product softmax of Eq. 1 (Sec. 3.1) with scale 1/sqrt(d_h);
//              the paper only names the proxy ("accumulated attention scores over an
//              observation window", Sec. 5.1; kernel 7 / window 32 in the baseline
//              hyper-parameter table), so the window/causal/sum/pool reading is the
//              conventional SnapKV one and is listed in the design notes.
//   hull     : PAVA projection of the marginal decreases onto a non-negative,
//              non-increasing sequence (Sec. 4.2, Eq. "marginal_gain"; App. A.2).
//   allocate : marginal-utility greedy == the B largest gains under the per-head prefix
//              constraint (Sec. 4.2 relaxed objective; App. A.2 "Optimality of greedy").
//   select   : top-b positions of a head by the proxy (Sec. 4.3 "Eviction"; M^pi(k) of
//              Sec. 3.2), ties by lower index (App. A.1 allows any fixed rule).
//   gather   : the retained index set I of Sec. 3.2 materialised as a packed cache.
//   curves   : utility-versus-budget curve of a proxy metric = running sum of the oracle
//              importance in the metric's ranking order (Sec. 3.2, Eq. "head_loss_def").
//   importance : the oracle importance of Sec. 4.1 (Eq. "oracle_importance"): the largest contribution
//              a cached position makes to the head output over K_max decode steps, attention weight
//              times the L2 norm of the projected value (App. E names the norm and an intra-layer
//              normalisation); readings for grouped queries and the normalisation in the design notes.
//   keydiff  : the second proxy metric the paper evaluates (Sec. 5.1, pi_2; App. E: recent window 1).  The paper
//              only names it (as a metric on the geometry of the key vectors); the formula restated here is the one of
//              the method's own publication (a key's score is the negated cosine similarity between the key and
//              the mean of all unit-normalised keys of its head), recorded as a reading in the design notes.
//   exact    : the allocation problem on the raw curves by the multiple-choice-knapsack
//              recursion (Sec. 4.2 mentions the exact solver as the comparison point).
//   deployment settings (App. E): attention sinks always ranked first; a minimum number of
//              tokens per head handed out before the greedy starts.  Both default to off.
//   profile  : offline profile = mean over calibration queries of the optimal local ratios
//              (Sec. 4.3, Eq. "calibration_avg"); online lookup and b = floor((1-r)*n)
//              (Sec. 4.3 "Online Execution").
//
// Pins (see tests, "-m not gpu"): softmax rows sum to one; closed form for identical
// keys; single-row case against a library softmax; pooling against a library max filter;
// PAVA against a library isotonic regression, a monotone-chain hull and the O(P^2)
// majorant definition; greedy against exhaustive search; selection against a full sort;
// uniform budgets against a library-op SnapKV; gather by byte equality; profile against a
// token-by-token greedy written in the test, the closed form for identical heads, the end
// points rho = 0 and 1, budget conservation and monotonicity in rho; lookup against a
// hand-worked example; curves against the pinned selection (importance mass of M^pi(k)), a
// library sort for the oracle metric, and closed forms; the exact solver against exhaustive
// search, against the greedy on concave curves, and between the greedy's raw and hull values;
// the oracle importance against a library softmax times a library vector norm (one decode step,
// identity projection), closed forms for identical keys, monotonicity in K_max, a dominant decode
// key, doubling under two identical grouped query heads, and unit mass per layer after normalisation;
// the KeyDiff score against library cosine-similarity and normalisation routines, closed forms
// (identical keys, one odd key out, two opposite groups), and invariance to rescaling single keys.
// No function here is "parity unpinned".
//
// Build: g++ -O2 -std=c++17 -ffp-contract=off -shared -fPIC lukv_oracle.cpp -o liblukv_oracle.so

#include <algorithm>
#include <cfloat>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <numeric>
#include <vector>

namespace {

// bf16 is the upper half of an IEEE binary32: widening is exact.
inline float bf16_bits_to_float(uint16_t b) {
  uint32_t u = static_cast<uint32_t>(b) << 16;
  float f;
  std::memcpy(&f, &u, sizeof f);
  return f;
}

// dtype 0: bf16 stored as uint16 bit patterns; dtype 1: fp32.
inline double load_elem(const void* base, int dtype, int64_t idx) {
  if (dtype == 0) return static_cast<double>(bf16_bits_to_float(static_cast<const uint16_t*>(base)[idx]));
  return static_cast<double>(static_cast<const float*>(base)[idx]);
}

inline size_t elem_size(int dtype) { return dtype == 0 ? 2 : 4; }

// Round a double to fp32 (nearest-even); magnitudes below FLT_MIN become +0, mirroring
// the flush-to-zero arithmetic of the device the oracle is compared with.
inline float to_f32_ftz(double x) {
  float f = static_cast<float>(x);
  if (std::fabs(f) < FLT_MIN) f = 0.0f;
  return f;
}

struct Dims {
  int S, L, H, G, d, T, w, kp, dtype, P;
  double scale;
  int N() const { return L * H; }
  int n() const { return T - w; }
};

// ---- score ---------------------------------------------------------------------------
// One KV head. q_head: [G][w][d] (the G query heads of this KV head are contiguous in
// the [H*G] axis), k_head: [T][d].
// Row r=(g,i) is the query at position n+i; it sees keys j <= n+i (causal, Eq. 1 applied
// at that position).  prob (optional): [G*w][T], masked entries 0.  raw_full (optional):
// [T] column sums over all rows, in double.
void score_head(const void* q_head, const void* k_head, int dtype, int G, int w, int d, int T,
                double scale, double* prob, double* raw_full) {
  const int n = T - w;
  std::vector<double> kd(static_cast<size_t>(T) * d);
  for (int64_t e = 0; e < static_cast<int64_t>(T) * d; ++e) kd[e] = load_elem(k_head, dtype, e);
  std::vector<double> qd(d), x(T);
  if (raw_full) std::fill(raw_full, raw_full + T, 0.0);
  for (int g = 0; g < G; ++g) {
    for (int i = 0; i < w; ++i) {
      const int r = g * w + i;
      for (int c = 0; c < d; ++c) qd[c] = load_elem(q_head, dtype, (static_cast<int64_t>(g) * w + i) * d + c);
      const int visible = n + i + 1;  // keys 0 .. n+i
      double m = -INFINITY;
      for (int j = 0; j < visible; ++j) {
        double acc = 0.0;
        const double* kj = &kd[static_cast<size_t>(j) * d];
        for (int c = 0; c < d; ++c) acc += qd[c] * kj[c];
        x[j] = scale * acc;
        if (x[j] > m) m = x[j];
      }
      double Z = 0.0;
      for (int j = 0; j < visible; ++j) Z += std::exp(x[j] - m);
      for (int j = 0; j < visible; ++j) {
        const double p = std::exp(x[j] - m) / Z;
        if (prob) prob[static_cast<size_t>(r) * T + j] = p;
        if (raw_full) raw_full[j] += p;
      }
      if (prob)
        for (int j = visible; j < T; ++j) prob[static_cast<size_t>(r) * T + j] = 0.0;
    }
  }
}

// Centred, stride-1 max filter of odd width kp over [0,n); the filter window is clipped
// at both ends (equivalently padded with -inf).
void max_pool(const double* raw, int n, int kp, double* pooled) {
  const int half = kp / 2;
  for (int j = 0; j < n; ++j) {
    const int lo = std::max(0, j - half), hi = std::min(n - 1, j + half);
    double best = raw[lo];
    for (int t = lo + 1; t <= hi; ++t) best = std::max(best, raw[t]);
    pooled[j] = best;
  }
}

// ---- hull ----------------------------------------------------------------------------
// PAVA on the P-1 increments of a utility curve U[0..P-1] (utility = L(0) - L(b), so its
// increments are the paper's marginal decreases of the loss).  Blocks are kept on a
// stack as [l, r) spans of curve points; a block's value is its mean increment
// (U[r]-U[l])/(r-l).  A new increment is pushed as its own block and merged with the
// block before it while that block's mean is <= the new one's (violating or tying the
// required non-increasing order).  Each segment's gain is its block mean clipped at 0.
void pava_gains(const float* U, int P, double* gains) {
  struct Block { int l, r; double mean; };
  std::vector<Block> st;
  st.reserve(P);
  for (int k = 0; k + 1 < P; ++k) {
    Block cur{k, k + 1, (static_cast<double>(U[k + 1]) - static_cast<double>(U[k])) / 1.0};
    while (!st.empty() && st.back().mean <= cur.mean) {
      cur.l = st.back().l;
      st.pop_back();
      cur.mean = (static_cast<double>(U[cur.r]) - static_cast<double>(U[cur.l])) / static_cast<double>(cur.r - cur.l);
    }
    st.push_back(cur);
  }
  for (const Block& b : st) {
    const double g = b.mean > 0.0 ? b.mean : 0.0;
    for (int k = b.l; k < b.r; ++k) gains[k] = g;
  }
}

// Capacity (tokens) of segment k of a head: the curve grid has step s = T/(P-1) tokens
// and only the n = T - w non-window positions can be bought.
inline int64_t seg_cap(int k, int64_t s, int64_t n) {
  int64_t c = n - static_cast<int64_t>(k) * s;
  if (c < 0) c = 0;
  if (c > s) c = s;
  return c;
}

struct Item { float gain; int k; int hid; int64_t cap; };

// Tokens of segment k of a head that are still for sale when the head's first f tokens are
// given to it up front (the minimum retention of App. E).
inline int64_t seg_cap_after_floor(int k, int64_t s, int64_t n, int64_t f) {
  const int64_t lo = std::max<int64_t>(static_cast<int64_t>(k) * s, f);
  const int64_t hi = std::min<int64_t>(static_cast<int64_t>(k + 1) * s, n);
  return hi > lo ? hi - lo : 0;
}

// ---- select --------------------------------------------------------------------------
// First b positions of the order (score descending, index ascending), emitted ascending.
// Attention sinks (App. E: sink size 4): the first n_sink positions rank before every other
// position whatever their score, so they are kept whenever the budget allows (b >= n_sink)
// and count towards it.
void select_head(const float* pooled, int n, int b, int n_sink, int32_t* kept) {
  std::vector<int32_t> order(n);
  std::iota(order.begin(), order.end(), 0);
  std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t c) {
    const bool sa = a < n_sink, sc = c < n_sink;
    if (sa != sc) return sa;
    if (sa) return false;  // both sinks: position order (stable)
    return pooled[a] > pooled[c];
  });
  std::vector<int32_t> top(order.begin(), order.begin() + b);
  std::sort(top.begin(), top.end());
  std::copy(top.begin(), top.end(), kept);
}

}  // namespace

extern "C" {

// Probability matrix of one head (for the row-sum pin). prob: [G*w][T] doubles.
void oracle_window_softmax(const void* q_head, const void* k_head, int dtype, int G, int w, int d, int T,
                           float scale, double* prob) {
  const double sc = scale != 0.0f ? static_cast<double>(scale) : 1.0 / std::sqrt(static_cast<double>(d));
  score_head(q_head, k_head, dtype, G, w, d, T, sc, prob, nullptr);
}

// One head: raw_full [T] doubles (may be null), pooled [n] floats (may be null).
void oracle_score_head(const void* q_head, const void* k_head, int dtype, int G, int w, int d, int T, int kp,
                       float scale, double* raw_full, float* pooled) {
  const double sc = scale != 0.0f ? static_cast<double>(scale) : 1.0 / std::sqrt(static_cast<double>(d));
  const int n = T - w;
  std::vector<double> raw(T), pl(n);
  score_head(q_head, k_head, dtype, G, w, d, T, sc, nullptr, raw.data());
  if (raw_full) std::copy(raw.begin(), raw.end(), raw_full);
  if (pooled) {
    max_pool(raw.data(), n, kp, pl.data());
    for (int j = 0; j < n; ++j) pooled[j] = to_f32_ftz(pl[j]);
  }
}

// All heads. q: [S][L][H*G][w][d], k: [S][L][H][T][d], scores: [S][L*H][n].
void oracle_score(const void* q, const void* k, int dtype, int S, int L, int H, int G, int d, int T, int w,
                  int kp, float scale, float* scores) {
  const int n = T - w;
  const size_t es = elem_size(dtype);
  for (int64_t u = 0; u < static_cast<int64_t>(S) * L * H; ++u) {
    const char* qh = static_cast<const char*>(q) + static_cast<size_t>(u) * G * w * d * es;
    const char* kh = static_cast<const char*>(k) + static_cast<size_t>(u) * T * d * es;
    oracle_score_head(qh, kh, dtype, G, w, d, T, kp, scale, nullptr, scores + u * n);
  }
}

// Stand-alone max-pool over [0,n) (pin: library max filter).
void oracle_max_pool(const double* raw, int n, int kp, double* pooled) { max_pool(raw, n, kp, pooled); }

// Hull gains of N curves. curves: [N][P] floats; gains_f64 (may be null): [N][P-1]
// doubles before the final rounding; gains_f32 (may be null): rounded once to fp32.
void oracle_hull(const float* curves, int N, int P, double* gains_f64, float* gains_f32) {
  std::vector<double> g(P - 1);
  for (int h = 0; h < N; ++h) {
    pava_gains(curves + static_cast<size_t>(h) * P, P, g.data());
    for (int k = 0; k + 1 < P; ++k) {
      if (gains_f64) gains_f64[static_cast<size_t>(h) * (P - 1) + k] = g[k];
      if (gains_f32) gains_f32[static_cast<size_t>(h) * (P - 1) + k] = static_cast<float>(g[k]);
    }
  }
}

// Greedy allocation. curves: [N][P]; budgets_in: [S] selectable tokens per sequence;
// budgets: [S][N]; offsets: [S*N+1] = exclusive scan of (budget + w) in head order
// u = q*N + hid.  Returns 0, or -1 when some B_q is outside [0, N*n].
// Items are all (hid,k) with non-zero capacity, ordered by (gain descending, k ascending,
// hid ascending); they are consumed in that order until B_q tokens are spent, the last
// one partially.
//
// floor_tokens f (App. E: no head is compressed beyond 99 %, i.e. keeps at least 1 % of its
// tokens): every head first receives its f highest-ranked tokens, the greedy then spends
// B_q - N*f on what is left.  f = 0 is the plain greedy.  Returns -1 also when B_q < N*f.
int oracle_allocate_floor(const float* curves, int N, int P, int T, int w, int S, const int64_t* budgets_in,
                          int64_t floor_tokens, int32_t* budgets, int32_t* offsets) {
  const int64_t n = T - w, s = T / (P - 1), f = floor_tokens;
  if (f < 0 || f > n) return -1;
  std::vector<float> g(static_cast<size_t>(N) * (P - 1));
  oracle_hull(curves, N, P, nullptr, g.data());
  std::vector<Item> items;
  for (int hid = 0; hid < N; ++hid)
    for (int k = 0; k + 1 < P; ++k) {
      const int64_t cap = f == 0 ? seg_cap(k, s, n) : seg_cap_after_floor(k, s, n, f);
      if (cap > 0) items.push_back(Item{g[static_cast<size_t>(hid) * (P - 1) + k], k, hid, cap});
    }
  std::sort(items.begin(), items.end(), [](const Item& a, const Item& b) {
    if (a.gain != b.gain) return a.gain > b.gain;
    if (a.k != b.k) return a.k < b.k;
    return a.hid < b.hid;
  });
  int64_t running = 0;
  offsets[0] = 0;
  for (int q = 0; q < S; ++q) {
    const int64_t B = budgets_in[q];
    if (B < static_cast<int64_t>(N) * f || B > static_cast<int64_t>(N) * n) return -1;
    std::vector<int64_t> b(N, f);
    int64_t left = B - static_cast<int64_t>(N) * f;
    for (const Item& it : items) {
      if (left == 0) break;
      const int64_t take = std::min(left, it.cap);
      b[it.hid] += take;
      left -= take;
    }
    for (int hid = 0; hid < N; ++hid) {
      budgets[static_cast<size_t>(q) * N + hid] = static_cast<int32_t>(b[hid]);
      running += b[hid] + w;
      offsets[static_cast<size_t>(q) * N + hid + 1] = static_cast<int32_t>(running);
    }
  }
  return 0;
}

int oracle_allocate(const float* curves, int N, int P, int T, int w, int S, const int64_t* budgets_in,
                    int32_t* budgets, int32_t* offsets) {
  return oracle_allocate_floor(curves, N, P, T, w, S, budgets_in, 0, budgets, offsets);
}

// Tokens every head keeps at least: ceil(min_keep * n), min_keep in [0,1] (App. E uses 0.01).
int64_t oracle_floor_tokens(float min_keep, int n) {
  const double f = std::ceil(static_cast<double>(min_keep) * static_cast<double>(n));
  return f < 0.0 ? 0 : (f > n ? n : static_cast<int64_t>(f));
}

// Offline profile aggregation (Sec. 4.3 "Profile Aggregation", Eq. "calibration_avg").
// curves: [Mq][N][P], one set of per-head utility curves per calibration query, taken on a
// calibration context of T tokens (n = T-w rankable).  ratios: [R] global compression
// ratios rho in [0,1].  For every query and every rho the relaxed problem is solved for the
// global budget B(rho) = floor((1-rho)*N*n); the query's optimal local ratio of head hid is
// r* = 1 - b_hid/n; the profile is the mean of r* over the queries.
// profile: [R][N], fp64 mean rounded once to fp32.  Returns 0, or -1 for a ratio outside [0,1].
// min_keep > 0 (App. E): every head keeps at least f = ceil(min_keep*n) tokens in every solution, and
// a grid ratio whose budget would fall below N*f is solved for N*f.
int oracle_profile_build_floor(const float* curves, int Mq, int N, int P, int T, int w, const float* ratios, int R,
                               float min_keep, float* profile) {
  const int64_t n = T - w;
  const int64_t f = oracle_floor_tokens(min_keep, static_cast<int>(n));
  std::vector<int64_t> B(R);
  for (int j = 0; j < R; ++j) {
    const double rho = static_cast<double>(ratios[j]);
    if (!(rho >= 0.0 && rho <= 1.0)) return -1;
    B[j] = static_cast<int64_t>(std::floor((1.0 - rho) * static_cast<double>(static_cast<int64_t>(N) * n)));
    if (B[j] < static_cast<int64_t>(N) * f) B[j] = static_cast<int64_t>(N) * f;
  }
  std::vector<double> acc(static_cast<size_t>(R) * N, 0.0);
  std::vector<int32_t> b(static_cast<size_t>(R) * N), off(static_cast<size_t>(R) * N + 1);
  for (int i = 0; i < Mq; ++i) {
    const float* ci = curves + static_cast<size_t>(i) * N * P;
    if (oracle_allocate_floor(ci, N, P, T, w, R, B.data(), f, b.data(), off.data()) != 0) return -1;
    for (size_t e = 0; e < acc.size(); ++e) acc[e] += 1.0 - static_cast<double>(b[e]) / static_cast<double>(n);
  }
  for (size_t e = 0; e < acc.size(); ++e) profile[e] = static_cast<float>(acc[e] / static_cast<double>(Mq));
  return 0;
}

int oracle_profile_build(const float* curves, int Mq, int N, int P, int T, int w, const float* ratios, int R,
                         float* profile) {
  return oracle_profile_build_floor(curves, Mq, N, P, T, w, ratios, R, 0.f, profile);
}

// Online lookup and budgeting (Sec. 4.3 "Online Execution", steps 1-2).  profile: [R][N] over
// the strictly ascending grid ratios[R]; sigma: [S] target global ratio of each sequence,
// inside [ratios[0], ratios[R-1]].  Lookup: the profile row at sigma; between two grid points
// the two neighbouring rows are interpolated linearly (at a grid point this is the row
// itself).  Budgeting: b = floor((1-r)*n) on the n = T-w rankable positions of the new
// context, all in fp64.  offsets: exclusive scan of (b + w) in head order.
// Returns 0, or -1 when a sigma lies outside the grid or the grid is not ascending.
// min_keep > 0: budgets below f = ceil(min_keep*n) are raised to f (App. E).
int oracle_profile_budgets_floor(const float* profile, const float* ratios, int R, int N, int T, int w,
                                 const float* sigma, int S, float min_keep, int32_t* budgets, int32_t* offsets) {
  const int64_t n = T - w;
  const int64_t f = oracle_floor_tokens(min_keep, static_cast<int>(n));
  for (int j = 0; j + 1 < R; ++j)
    if (!(ratios[j] < ratios[j + 1])) return -1;
  int64_t running = 0;
  offsets[0] = 0;
  for (int q = 0; q < S; ++q) {
    const float sg = sigma[q];
    if (!(sg >= ratios[0] && sg <= ratios[R - 1])) return -1;
    int j = 0;
    while (j + 1 < R && ratios[j + 1] <= sg) ++j;  // largest j with ratios[j] <= sigma
    const int j1 = j + 1 < R ? j + 1 : j;
    const double t = j1 == j ? 0.0
                             : (static_cast<double>(sg) - static_cast<double>(ratios[j])) /
                                   (static_cast<double>(ratios[j1]) - static_cast<double>(ratios[j]));
    for (int hid = 0; hid < N; ++hid) {
      const double r0 = static_cast<double>(profile[static_cast<size_t>(j) * N + hid]);
      const double r1 = static_cast<double>(profile[static_cast<size_t>(j1) * N + hid]);
      const double r = r0 + (r1 - r0) * t;
      double bf = std::floor((1.0 - r) * static_cast<double>(n));
      if (bf < 0.0) bf = 0.0;
      if (bf > static_cast<double>(n)) bf = static_cast<double>(n);
      int64_t bq = static_cast<int64_t>(bf);
      if (bq < f) bq = f;
      budgets[static_cast<size_t>(q) * N + hid] = static_cast<int32_t>(bq);
      running += bq + w;
      offsets[static_cast<size_t>(q) * N + hid + 1] = static_cast<int32_t>(running);
    }
  }
  return 0;
}

int oracle_profile_budgets(const float* profile, const float* ratios, int R, int N, int T, int w,
                           const float* sigma, int S, int32_t* budgets, int32_t* offsets) {
  return oracle_profile_budgets_floor(profile, ratios, R, N, T, w, sigma, S, 0.f, budgets, offsets);
}

// Top-b of one head. pooled: [n]; kept: [b], ascending positions.
void oracle_select(const float* pooled, int n, int b, int32_t* kept) { select_head(pooled, n, b, 0, kept); }
void oracle_select_sink(const float* pooled, int n, int b, int n_sink, int32_t* kept) {
  select_head(pooled, n, b, n_sink, kept);
}

// Exact solution of the allocation problem (Sec. 4.2, Eq. "combinatorial_optimization": maximise
// the summed utility -- minimise the summed loss -- over integer budgets with sum b = B), on the
// curves as given (no relaxation), by dynamic programming over the heads: the classic
// multiple-choice-knapsack recursion f_h(x) = max_b f_{h-1}(x-b) + U_h(b).  Token-resolution
// curves only (P = T+1, point b = utility of keeping b tokens, 0 <= b <= n).  fp64.
// budgets: [S][N] one optimal solution (the smallest b on ties, heads taken last to first);
// values: [S] the optimum.  Returns 0, or -1 for s != 1 or a budget outside [0, N*n].
int oracle_exact_allocate(const float* curves, int N, int P, int T, int w, int S, const int64_t* budgets_in,
                          int32_t* budgets, double* values) {
  const int64_t n = T - w;
  if (P != T + 1) return -1;
  const double ninf = -std::numeric_limits<double>::infinity();
  for (int q = 0; q < S; ++q) {
    const int64_t B = budgets_in[q];
    if (B < 0 || B > static_cast<int64_t>(N) * n) return -1;
    std::vector<double> f(B + 1, ninf), g(B + 1);
    std::vector<int32_t> choice(static_cast<size_t>(N) * (B + 1));
    f[0] = 0.0;
    for (int h = 0; h < N; ++h) {
      const float* U = curves + static_cast<size_t>(h) * P;
      for (int64_t x = 0; x <= B; ++x) {
        double best = ninf;
        int32_t arg = 0;
        const int64_t bmax = std::min<int64_t>(x, n);
        for (int64_t b = 0; b <= bmax; ++b) {
          const double v = f[x - b] + static_cast<double>(U[b]);
          if (v > best) {
            best = v;
            arg = static_cast<int32_t>(b);
          }
        }
        g[x] = best;
        choice[static_cast<size_t>(h) * (B + 1) + x] = arg;
      }
      f.swap(g);
    }
    values[q] = f[B];
    int64_t x = B;
    for (int h = N - 1; h >= 0; --h) {
      const int32_t b = choice[static_cast<size_t>(h) * (B + 1) + x];
      budgets[static_cast<size_t>(q) * N + h] = b;
      x -= b;
    }
  }
  return 0;
}

// Oracle importance (Sec. 4.1, Eq. "oracle_importance"):  I_j = max_{k=1..K_max} A_{k,j} * || v_j W_O ||_2.
//   A_{k,j}: attention weight (Eq. 1) of the query of decode step k on cached position j.  The softmax of step k
//            runs over the T cached positions and, when decode keys are given, over the keys of decode steps
//            1..k as well (causal, the step's own key included).
//   grouped queries: a KV head is read by G query heads, each with its own slice of the output projection;
//            the importance of a cached position adds their contributions before the maximum over the steps:
//            I_j = max_k sum_g A_{g,k,j} * || v_j W_O^(g) ||_2   (G = 1 is the paper's formula as printed).
//   normalisation (App. E, "intra-layer normalisation"): every layer's values are divided by their sum over the
//            layer's heads and rankable positions, so that each layer carries unit mass.
// q_dec [S][L][H*G][Kmax][d], k, v [S][L][H][T][d], k_dec [S][L][H][Kmax][d] or null, w_o [L][H*G][d][Dm];
// out importance [S][L*H][T-w] fp32 (window positions are always kept and never enter a loss).
void oracle_importance(const void* q_dec, const void* k, const void* v, const void* k_dec, const void* w_o, int dtype,
                       int S, int L, int H, int G, int d, int T, int w, int Kmax, int Dm, float scale_in,
                       int normalize, float* importance) {
  const int n = T - w;
  const double scale = scale_in > 0.f ? static_cast<double>(scale_in) : 1.0 / std::sqrt(static_cast<double>(d));
  std::vector<double> imp(static_cast<size_t>(S) * L * H * n);
  std::vector<double> vnorm(static_cast<size_t>(G) * T), x(static_cast<size_t>(T) + Kmax), s(T), y(Dm);
  for (int q = 0; q < S; ++q)
    for (int l = 0; l < L; ++l)
      for (int h = 0; h < H; ++h) {
        const int64_t u = (static_cast<int64_t>(q) * L + l) * H + h;
        const int64_t kbase = u * T * d, dbase = u * Kmax * d;
        // || v_j W_O^(g) ||_2
        for (int g = 0; g < G; ++g) {
          const int64_t wbase = (static_cast<int64_t>(l) * H * G + h * G + g) * d * Dm;
          for (int j = 0; j < T; ++j) {
            std::fill(y.begin(), y.end(), 0.0);
            for (int c = 0; c < d; ++c) {
              const double vc = load_elem(v, dtype, kbase + static_cast<int64_t>(j) * d + c);
              for (int m = 0; m < Dm; ++m) y[m] += vc * load_elem(w_o, dtype, wbase + static_cast<int64_t>(c) * Dm + m);
            }
            double ss = 0.0;
            for (int m = 0; m < Dm; ++m) ss += y[m] * y[m];
            vnorm[static_cast<size_t>(g) * T + j] = std::sqrt(ss);
          }
        }
        double* out = imp.data() + u * n;
        std::fill(out, out + n, 0.0);
        for (int kk = 0; kk < Kmax; ++kk) {
          std::fill(s.begin(), s.end(), 0.0);
          for (int g = 0; g < G; ++g) {
            const int64_t qbase = (((static_cast<int64_t>(q) * L + l) * H * G + h * G + g) * Kmax + kk) * d;
            const int visible = T + (k_dec ? kk + 1 : 0);
            double mx = -std::numeric_limits<double>::infinity();
            for (int j = 0; j < visible; ++j) {
              double dot = 0.0;
              for (int c = 0; c < d; ++c) {
                const double kc = j < T ? load_elem(k, dtype, kbase + static_cast<int64_t>(j) * d + c)
                                        : load_elem(k_dec, dtype, dbase + static_cast<int64_t>(j - T) * d + c);
                dot += load_elem(q_dec, dtype, qbase + c) * kc;
              }
              x[j] = dot * scale;
              mx = std::max(mx, x[j]);
            }
            double Z = 0.0;
            for (int j = 0; j < visible; ++j) Z += std::exp(x[j] - mx);
            for (int j = 0; j < T; ++j) s[j] += std::exp(x[j] - mx) / Z * vnorm[static_cast<size_t>(g) * T + j];
          }
          for (int j = 0; j < n; ++j) out[j] = std::max(out[j], s[j]);
        }
      }
  if (normalize) {
    for (int q = 0; q < S; ++q)
      for (int l = 0; l < L; ++l) {
        double* base = imp.data() + (static_cast<int64_t>(q) * L + l) * H * n;
        double total = 0.0;
        for (int64_t i = 0; i < static_cast<int64_t>(H) * n; ++i) total += base[i];
        if (total > 0.0)
          for (int64_t i = 0; i < static_cast<int64_t>(H) * n; ++i) base[i] /= total;
      }
  }
  for (size_t i = 0; i < imp.size(); ++i) importance[i] = to_f32_ftz(imp[i]);
}


// KeyDiff proxy (pi_2 of Sec. 5.1; formula from the method's own publication, see the header):
//   u_j = k_j / max(||k_j||, eps),   a = (1/T) sum_{j<T} u_j   (all T cached keys of the head, window included),
//   score_j = - <k_j, a> / (max(||k_j||, eps) * max(||a||, eps)),   eps = 1e-8,   for the n = T-w rankable positions.
// Keys far from the head's mean key direction score high and are kept.  k [heads][T][d]; out [heads][T-w] fp32.
void oracle_keydiff(const void* k, int dtype, int heads, int T, int w, int d, float* scores) {
  const int n = T - w;
  const double eps = 1e-8;
  std::vector<double> anchor(d), norm(T);
  for (int u = 0; u < heads; ++u) {
    const int64_t base = static_cast<int64_t>(u) * T * d;
    std::fill(anchor.begin(), anchor.end(), 0.0);
    for (int j = 0; j < T; ++j) {
      double ss = 0.0;
      for (int c = 0; c < d; ++c) {
        const double x = load_elem(k, dtype, base + static_cast<int64_t>(j) * d + c);
        ss += x * x;
      }
      norm[j] = std::max(std::sqrt(ss), eps);
      for (int c = 0; c < d; ++c) anchor[c] += load_elem(k, dtype, base + static_cast<int64_t>(j) * d + c) / norm[j];
    }
    double an = 0.0;
    for (int c = 0; c < d; ++c) {
      anchor[c] /= static_cast<double>(T);
      an += anchor[c] * anchor[c];
    }
    an = std::max(std::sqrt(an), eps);
    for (int j = 0; j < n; ++j) {
      double dot = 0.0;
      for (int c = 0; c < d; ++c) dot += load_elem(k, dtype, base + static_cast<int64_t>(j) * d + c) * anchor[c];
      scores[static_cast<int64_t>(u) * n + j] = static_cast<float>(-dot / (norm[j] * an));
    }
  }
}


// Utility-versus-budget curves of a proxy metric (Sec. 3.2: M^pi(k) is the set of the first k
// positions when ranked by pi; Eq. "head_loss_def": the eviction loss of a retained set is the
// oracle importance mass outside it).  U(k) = L(empty) - L(M^pi(k)) is the importance mass of
// the k highest-ranked positions, i.e. the running sum of the importance in ranking order.
// scores, importance: [heads][n] over the rankable positions; curves: [heads][P], point k =
// U(min(k*s, n)), s = T/(P-1); running sum in fp64, each point rounded once to fp32.
// Ranking as in the selection: sinks first, score descending, ties by lower position.
void oracle_build_curves(const float* scores, const float* importance, int heads, int T, int w, int P, int n_sink,
                         float* curves) {
  const int n = T - w, s = T / (P - 1);
  std::vector<int32_t> order(n);
  std::vector<double> cum(n + 1);
  for (int64_t u = 0; u < heads; ++u) {
    // the ranking of select_head, kept in ranking order
    std::iota(order.begin(), order.end(), 0);
    const float* sc = scores + u * n;
    std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t c) {
      const bool sa = a < n_sink, sb = c < n_sink;
      if (sa != sb) return sa;
      if (sa) return false;
      return sc[a] > sc[c];
    });
    cum[0] = 0.0;
    for (int i = 0; i < n; ++i) cum[i + 1] = cum[i] + static_cast<double>(importance[u * n + order[i]]);
    for (int k = 0; k < P; ++k) {
      const int64_t b = std::min<int64_t>(static_cast<int64_t>(k) * s, n);
      curves[u * P + k] = static_cast<float>(cum[b]);
    }
  }
}

// Selection + gather for all heads. scores: [S*N][n]; budgets: [S*N]; offsets: [S*N+1];
// k,v: [S*N][T][d]; k_out,v_out: [rows][d]; kept_idx: [rows].  For head u the packed rows
// [off, off+b) hold the kept positions in ascending order and rows [off+b, off+b+w) hold
// the window positions n..T-1.
void oracle_select_gather_sink(const float* scores, const int32_t* budgets, const int32_t* offsets, const void* k,
                               const void* v, int dtype, int heads, int T, int w, int d, int n_sink, void* k_out,
                               void* v_out, int32_t* kept_idx) {
  const int n = T - w;
  const size_t row = static_cast<size_t>(d) * elem_size(dtype);
  for (int64_t u = 0; u < heads; ++u) {
    const int b = budgets[u];
    int32_t* kept = kept_idx + offsets[u];
    select_head(scores + u * n, n, b, n_sink, kept);
    for (int i = 0; i < w; ++i) kept[b + i] = n + i;
    for (int t = 0; t < b + w; ++t) {
      const size_t src = (static_cast<size_t>(u) * T + kept[t]) * row;
      const size_t dst = (static_cast<size_t>(offsets[u]) + t) * row;
      std::memcpy(static_cast<char*>(k_out) + dst, static_cast<const char*>(k) + src, row);
      std::memcpy(static_cast<char*>(v_out) + dst, static_cast<const char*>(v) + src, row);
    }
  }
}

void oracle_select_gather(const float* scores, const int32_t* budgets, const int32_t* offsets, const void* k,
                          const void* v, int dtype, int heads, int T, int w, int d, void* k_out, void* v_out,
                          int32_t* kept_idx) {
  oracle_select_gather_sink(scores, budgets, offsets, k, v, dtype, heads, T, w, d, 0, k_out, v_out, kept_idx);
}

// The whole path: allocate (hull + greedy) and score are independent; selection needs
// both; gather follows.  scores_out (may be null): [S*N][n] pooled scores.
// n_sink, min_keep: the deployment settings of App. E (0, 0 switches them off).
int oracle_compress_ext(const void* q, const void* k, const void* v, const float* curves, const int64_t* budgets_in,
                        int dtype, int S, int L, int H, int G, int d, int T, int w, int kp, int P, float scale,
                        int n_sink, float min_keep, void* k_out, void* v_out, int32_t* kept_idx, int32_t* budgets,
                        int32_t* offsets, float* scores_out) {
  const int N = L * H, n = T - w;
  if (oracle_allocate_floor(curves, N, P, T, w, S, budgets_in, oracle_floor_tokens(min_keep, n), budgets, offsets) != 0)
    return -1;
  std::vector<float> local;
  float* sc = scores_out;
  if (!sc) {
    local.resize(static_cast<size_t>(S) * N * n);
    sc = local.data();
  }
  oracle_score(q, k, dtype, S, L, H, G, d, T, w, kp, scale, sc);
  oracle_select_gather_sink(sc, budgets, offsets, k, v, dtype, S * N, T, w, d, n_sink, k_out, v_out, kept_idx);
  return 0;
}

int oracle_compress(const void* q, const void* k, const void* v, const float* curves, const int64_t* budgets_in,
                    int dtype, int S, int L, int H, int G, int d, int T, int w, int kp, int P, float scale,
                    void* k_out, void* v_out, int32_t* kept_idx, int32_t* budgets, int32_t* offsets,
                    float* scores_out) {
  return oracle_compress_ext(q, k, v, curves, budgets_in, dtype, S, L, H, G, d, T, w, kp, P, scale, 0, 0.f, k_out, v_out,
                             kept_idx, budgets, offsets, scores_out);
}

}  // extern "C"
