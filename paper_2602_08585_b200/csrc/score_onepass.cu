// Stage (a) on the 5th-generation tensor cores (bf16, head_dim 128), one sweep over the keys:
// every window logit of Eq. 1 (Sec. 3.1) is computed once and goes through one exp2.
//
// A row's softmax normaliser needs every key of the head before any probability is final, and the
// score of a key sums the probabilities of all M = G*w rows.  This kernel therefore parks the
// exponentials in tensor memory until the row's log-sum-exp is known:
//   phase 1  D[query row][key] = Q K^T by tcgen05.mma into TMEM.  A thread owns one query row,
//            replaces the logits of its row by E = exp2(x*scale - ref) in place (ref: a per-row,
//            per-tile reference close to the tile's row maximum), and publishes the tile's row
//            log-sum-exp, ref + log2(sum E), as one float per (row, key tile)
//   fold     the row log-sum-exp over all key tiles of the head; row r is folded by the CTA that
//            owns work item r mod (items per head), so the folds of a head run in parallel
//   phase 2  score[key] = sum_r E[r][key] * exp2(ref_r - lse_r): the rows are TMEM lanes, so this
//            is a reduction across lanes.  The 16x256b load shape hands each thread four rows of
//            a column pair, which are combined with FMAs; three shuffle rounds finish the
//            reduction inside a warp and the four warps of a quad are added through shared memory.
// TMEM (512 columns) holds two work items, so phase 1 of item k+1 runs while the log-sum-exp of
// item k's head is on its way; a head's exponentials occupy (key tiles x 128 x MT) columns spread
// over the CTAs, which bounds the context length this kernel takes (the two-sweep kernel covers
// the rest).
//
// Work item = (head, MT==1: two key tiles, one per epilogue quad | MT==2: one key tile, one block
// of 128 query rows per quad).  Items are dealt round-robin to a cooperative grid of at most one
// CTA per SM; a head's items must not outnumber the CTAs.
// Warps: 8 epilogue (two quads; a warp may only touch the TMEM lanes 32*(warp%4)..+31), TMA
// producer, MMA issuer and TMEM owner, fold warp, log-sum-exp prefetch warp.
// Every wait is bounded; a wait that runs out raises the CTA's abort flag and stores
// LUKV_ERR_TIMEOUT to the status word; the CTA then skips the remaining work and tears down.
#include "tc_ptx.cuh"

namespace lukv {
namespace {

constexpr uint32_t kSentinel = 0xFFFFFFFFu;  // "not published yet" in the partials (a NaN pattern no result has)

template <int MT>
struct OnePlan {
  static constexpr int kEpiWarps = 8;
  static constexpr int kThreads = (kEpiWarps + 4) * 32;
  static constexpr int kItemTiles = MT == 1 ? 2 : 1;   // key tiles per work item
  static constexpr int kStages = MT == 1 ? 4 : 2;      // key-tile ring
  static constexpr int kQSlots = 2;
  static constexpr int kQBytes = MT * kStageBytes;     // [half][MT*128 rows][128 B]
  static constexpr int kKOff = kQSlots * kQBytes;
  static constexpr int kBarOff = kKOff + kStages * kStageBytes;
  // barriers: kfull[kStages], kempty[kStages], qfull[2], qempty[2], tfull[4], tempty[4], lsefull[2], lseempty[2]
  static constexpr int kBarKFull = 0, kBarKEmpty = kStages, kBarQFull = 2 * kStages, kBarQEmpty = kBarQFull + kQSlots,
                       kBarTFull = kBarQEmpty + kQSlots, kBarTEmpty = kBarTFull + 4, kBarLseFull = kBarTEmpty + 4,
                       kBarLseEmpty = kBarLseFull + 2, kNumBars = kBarLseEmpty + 2;
  static constexpr int kMiscOff = (kBarOff + kNumBars * 8 + 15) & ~15;  // tmem base, abort flag, per-quad copies of it
  static constexpr int kPartOff = kMiscOff + 32;            // [2][8 warps][128] column sums over a warp's 32 rows
  static constexpr int kLseOff = kPartOff + 2 * 8 * 128 * 4;  // [2 slots][256] -lse of the items in flight
  static constexpr int kTotal = kLseOff + 2 * 256 * 4 + 1024;  // + slack for the 1024-byte alignment
  static_assert(kTotal <= 232448, "exceeds the shared memory of one CTA");
};

struct OneArgs {
  float* stats;        // [heads][M][tiles_pad] log-sum-exp of (row, key tile), exp2 domain; all-ones bits at launch
  float* lse;          // [heads][128*MT] (row log-sum-exp, tag); zero at launch
  float* raw;          // out: [heads][n] un-pooled scores
  int32_t* dev_status;
  int M, T, w, n;
  int head0, nheads;   // heads [head0, head0+nheads) are scored by this launch
  int items_per_head, tiles_T, tiles_pad;
  float scale_log2;
  uint32_t spin_limit; // iterations a wait may take
  int drop_item;       // test hook: the partials of this work item are not published (-1: none)
};

struct Item {
  int u;       // head
  int c;       // item of the head
  int tile0;   // first key tile
  int ntiles;  // 1 or 2 (MT == 1), 1 (MT == 2)
  int index;   // item number of the launch
};

template <int MT>
__device__ __forceinline__ Item make_item(int k, const OneArgs& a) {
  Item it;
  it.index = (int)blockIdx.x + k * (int)gridDim.x;
  const int hu = it.index / a.items_per_head;
  it.c = it.index - hu * a.items_per_head;
  it.u = a.head0 + hu;
  it.tile0 = it.c * OnePlan<MT>::kItemTiles;
  it.ntiles = min(OnePlan<MT>::kItemTiles, a.tiles_T - it.tile0);
  return it;
}

// Which exp2 pairs of a 32-element chunk go to the FMA pipe instead of the special-function unit.
#ifndef LUKV_ONE_POLY_SEL
#define LUKV_ONE_POLY_SEL(i) ((((i) >> 2) & 3) == 0)
#endif

// Phase 1, 32 columns (keys jbase..jbase+31) of one query row.  (m, l): reference and sum of exp2(x - m)
// over the keys of the tile seen so far.  The chunk's exponentials are left in e[], relative to the m
// valid on return; `scale_prev` is the factor by which the tile's earlier chunks must be multiplied
// (1 unless the reference moved).
// The common path evaluates the chunk against the current reference and accepts the result while the
// chunk sum stays in a safe range; otherwise (first visible chunk, or a key far above the reference)
// the reference becomes the exact chunk maximum.  Either way m never exceeds the row's maximum, so an
// exponential that underflows here belongs to a probability below 2^-126.
template <bool MASKED>
__device__ __forceinline__ void p1_chunk(const float (&v)[32], int jbase, int lim, float scale_log2, float& m, float& l,
                                         float (&e)[32], float& scale_prev) {
  float x[32];
#pragma unroll
  for (int i = 0; i < 32; ++i) x[i] = (!MASKED || jbase + i <= lim) ? v[i] : -INFINITY;
  scale_prev = 1.f;
  if (m != -INFINITY) {
    const uint64_t sc2 = pack2(scale_log2, scale_log2), nm2 = pack2(-m, -m);
    uint64_t acc0 = 0ull, acc1 = 0ull;
    float pmax = -INFINITY;  // largest logit that went through the polynomial (it has no overflow of its own)
#pragma unroll
    for (int i = 0; i < 32; i += 4) {
      const uint64_t e0 = ex2_pair(ffma2(pack2(x[i], x[i + 1]), sc2, nm2));
      uint64_t e1;
      if (LUKV_ONE_POLY_SEL(i)) {
        pmax = fmaxf(pmax, fmaxf(x[i + 2], x[i + 3]));
        e1 = ex2_poly_pair<false>(ffma2(pack2(x[i + 2], x[i + 3]), sc2, nm2));
      } else {
        e1 = ex2_pair(ffma2(pack2(x[i + 2], x[i + 3]), sc2, nm2));
      }
      acc0 = fadd2(acc0, e0);
      acc1 = fadd2(acc1, e1);
      unpack2(e0, e[i], e[i + 1]);
      unpack2(e1, e[i + 2], e[i + 3]);
    }
    const float cs = sum4(acc0, acc1);
    if (cs <= 1e12f && fmaf(pmax, scale_log2, -m) <= 100.f) {  // false for inf and NaN
      l += cs;
      return;
    }
  }
  float cmax = x[0];
#pragma unroll
  for (int i = 1; i < 32; ++i) cmax = fmaxf(cmax, x[i]);
  const float mn = fmaxf(m, cmax * scale_log2);  // scale > 0
  if (mn == -INFINITY) {  // no visible key in the tile so far
#pragma unroll
    for (int i = 0; i < 32; ++i) e[i] = 0.f;
    return;
  }
  if (mn > m) {
    if (m != -INFINITY) {
      scale_prev = ex2(m - mn);
      l *= scale_prev;
    }
    m = mn;
  }
  float a0 = 0.f, a1 = 0.f;
#pragma unroll
  for (int i = 0; i < 32; i += 2) {
    e[i] = ex2(fmaf(x[i], scale_log2, -m));
    e[i + 1] = ex2(fmaf(x[i + 1], scale_log2, -m));
    a0 += e[i];
    a1 += e[i + 1];
  }
  l += a0 + a1;
}

// Phase 1 of one accumulator (128 keys of this thread's query row): logits -> exponentials in place.
template <bool MASKED>
__device__ __forceinline__ void p1_tile(uint32_t tcol, int j0, int lim, float scale_log2, float& m, float& l) {
  float va[32], vb[32], e[32];
  tmem_ld32(tcol, va);
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    float (&cur)[32] = (c & 1) ? vb : va;
    float (&nxt)[32] = (c & 1) ? va : vb;
    tmem_ld_wait(cur);
    if (c + 1 < 4) tmem_ld32(tcol + 32 * (c + 1), nxt);
    float f;
    p1_chunk<MASKED>(cur, j0 + 32 * c, lim, scale_log2, m, l, e, f);
    __syncwarp();
    if (c > 0 && __any_sync(0xffffffffu, f != 1.f)) {
      // the reference moved: bring the chunks stored so far to the new one (rare; all lanes take part
      // because the TMEM accesses are warp-wide, lanes whose reference stayed multiply by 1)
      if (c + 1 < 4) tmem_ld_wait(nxt);
      tmem_st_wait();
      float t[32];
      for (int cc = 0; cc < c; ++cc) {
        tmem_ld32(tcol + 32 * cc, t);
        tmem_ld_wait(t);
#pragma unroll
        for (int i = 0; i < 32; ++i) t[i] *= f;
        tmem_st32(tcol + 32 * cc, t);
        tmem_st_wait();
      }
    }
    tmem_st32(tcol + 32 * c, e);
  }
  tmem_st_wait();
}

__device__ __forceinline__ uint64_t sel64(bool p, uint64_t a, uint64_t b) { return p ? a : b; }

// One round of the reduce-scatter over the lanes that differ in bit `bit` of the lane index: a lane with
// the bit clear keeps the lower half of the pairs and receives the partner's lower half, and vice versa.
template <int HALF>
__device__ __forceinline__ void butterfly_round(uint64_t (&p)[8], bool upper, int bit) {
#pragma unroll
  for (int i = 0; i < HALF; ++i) {
    const uint64_t send = sel64(upper, p[i], p[i + HALF]);
    const uint64_t keep = sel64(upper, p[i + HALF], p[i]);
    const uint64_t recv = __shfl_xor_sync(0xffffffffu, (unsigned long long)send, bit);
    p[i] = fadd2(keep, recv);
  }
}

// acc[i] (+)= rows (t/4, t/4+8) of a 16-lane load times their factors, for the 8 column pairs of the load
__device__ __forceinline__ void p2_fma(uint64_t (&acc)[8], const float (&v)[32], float ca, float cb, bool first) {
  const uint64_t ca2 = pack2(ca, ca), cb2 = pack2(cb, cb);
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const uint64_t lo = pack2(v[4 * i], v[4 * i + 1]);
    const uint64_t hi = pack2(v[4 * i + 2], v[4 * i + 3]);
    // products below 2^-126 flush to zero (ftz): they are below the resolution of the scores
    uint64_t s = first ? ffma2(lo, ca2, 0ull) : ffma2(lo, ca2, acc[i]);
    acc[i] = ffma2(hi, cb2, s);
  }
}

template <int MT>
__global__ void __launch_bounds__(OnePlan<MT>::kThreads, 1)
    score_onepass_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap k_map,
                         const OneArgs a) {
  using P = OnePlan<MT>;
  constexpr int kStages = P::kStages;
  constexpr int kEpiWarps = P::kEpiWarps;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sbase = smem_u32(smem);
  const uint32_t q_s = sbase;
  const uint32_t k_s = sbase + P::kKOff;
  const uint32_t bars = sbase + P::kBarOff;
  auto bar = [&](int first, int i) { return bars + 8u * (uint32_t)(first + i); };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + P::kMiscOff);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + P::kMiscOff + 4);
  volatile int* quad_abort = reinterpret_cast<volatile int*>(smem + P::kMiscOff + 8);  // [2][2]
  float* part_s = reinterpret_cast<float*>(smem + P::kPartOff);  // [2][8][128]
  float* nlse_s = reinterpret_cast<float*>(smem + P::kLseOff);   // [2][256]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int total_items = a.nheads * a.items_per_head;
  const int K = (total_items - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;  // items of this CTA (>= 1)
  const uint32_t limit = a.spin_limit;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(bar(P::kBarKFull, s), 1);
      mbar_init(bar(P::kBarKEmpty, s), 1);
    }
    for (int s = 0; s < P::kQSlots; ++s) {
      mbar_init(bar(P::kBarQFull, s), 1);
      mbar_init(bar(P::kBarQEmpty, s), 1);
    }
    for (int b = 0; b < 4; ++b) {
      mbar_init(bar(P::kBarTFull, b), 1);
      mbar_init(bar(P::kBarTEmpty, b), 4);  // the four warps of the buffer's quad
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(bar(P::kBarLseFull, s), 1);
      mbar_init(bar(P::kBarLseEmpty, s), kEpiWarps);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kEpiWarps + 1) tmem_alloc(smem_u32((const void*)tmem_slot), 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == kEpiWarps) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      const uint64_t keep = l2_policy_evict_last();
      uint32_t tt = 0;
      for (int k = 0; k < K; ++k) {
        const Item it = make_item<MT>(k, a);
        const uint32_t slot = k & 1;
        if (!mbar_wait(bar(P::kBarQEmpty, slot), ((k >> 1) & 1) ^ 1, abort_flag, a.dev_status, limit)) break;
        mbar_expect_tx(bar(P::kBarQFull, slot), P::kQBytes);
        const uint32_t qd = q_s + slot * P::kQBytes;
        // the query tiles are read again by every item of the head: ask L2 to keep them
        for (int h = 0; h < 2; ++h)
          for (int mt = 0; mt < MT; ++mt)
            tma_load_2d_hint(qd + h * (MT * kHalfBytes) + mt * kHalfBytes, &q_map, bar(P::kBarQFull, slot), h * 64,
                             it.u * a.M + mt * 128, keep);
        bool ok = true;
        for (int t = 0; t < it.ntiles; ++t, ++tt) {
          const uint32_t s = tt % kStages, ph = (tt / kStages) & 1;
          if (!(ok = mbar_wait(bar(P::kBarKEmpty, s), ph ^ 1, abort_flag, a.dev_status, limit))) break;
          mbar_expect_tx(bar(P::kBarKFull, s), kStageBytes);
          const int row = it.u * a.T + (it.tile0 + t) * kTileKeys;
          const uint32_t dst = k_s + s * kStageBytes;
          tma_load_2d(dst, &k_map, bar(P::kBarKFull, s), 0, row);
          tma_load_2d(dst + kHalfBytes, &k_map, bar(P::kBarKFull, s), 64, row);
        }
        if (!ok) break;
      }
    }
  } else if (warp == kEpiWarps + 1) {
    // ---------------- MMA issuer ----------------
    // Accumulator (slot, q) = TMEM columns (2*slot + q)*128.  Its barriers complete once per item that
    // uses the slot whether or not the item has work for quad q, so every parity follows from the item
    // number alone.
    if (lane == 0) {
      constexpr uint32_t idesc = instr_desc_bf16(128, kTileKeys);
      uint32_t tt = 0;
      for (int k = 0; k < K; ++k) {
        const Item it = make_item<MT>(k, a);
        const uint32_t slot = k & 1, par = (k >> 1) & 1;
        const uint32_t qd = q_s + slot * P::kQBytes;
        bool ok = mbar_wait(bar(P::kBarQFull, slot), par, abort_flag, a.dev_status, limit);
        if (!ok) break;
        for (int q = 0; q < 2; ++q) {
          const uint32_t buf = 2 * slot + q;
          const bool active = MT == 2 || q < it.ntiles;
          if (active) {
            if (!(ok = mbar_wait(bar(P::kBarTEmpty, buf), par ^ 1, abort_flag, a.dev_status, limit))) break;
            const uint32_t s = tt % kStages, ph = (tt / kStages) & 1;
            if (MT == 1 || q == 0)
              if (!(ok = mbar_wait(bar(P::kBarKFull, s), ph, abort_flag, a.dev_status, limit))) break;
            tc_fence_after();
            const uint32_t kt = k_s + s * kStageBytes;
            const uint32_t d_tmem = tmem_base + buf * 128;
            const int mt = MT == 2 ? q : 0;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
              const int h = ks >> 2, sub = ks & 3;
              const uint64_t da = smem_desc_sw128(qd + h * (MT * kHalfBytes) + mt * kHalfBytes) + (uint64_t)(sub * 2);
              const uint64_t db = smem_desc_sw128(kt + h * kHalfBytes) + (uint64_t)(sub * 2);
              umma_bf16(d_tmem, da, db, idesc, ks > 0);
            }
            if (MT == 1 || q == 1) {
              umma_commit(bar(P::kBarKEmpty, s));  // the stage may be refilled once these MMAs have read it
              ++tt;
            }
          }
          umma_commit(bar(P::kBarTFull, buf));  // the accumulator is complete (or the item leaves it unused)
        }
        if (!ok) break;
        umma_commit(bar(P::kBarQEmpty, slot));
      }
    }
  } else if (warp == kEpiWarps + 2) {
    // ---------------- fold warp ----------------
    // Item c of a head folds the rows r = c, c + items_per_head, ... of that head: it waits until every
    // key tile's value for the row is there (the partials start as all-ones bit patterns), adds them as
    // lse = max + log2(sum exp2(v - max)) in a fixed order, and stores (lse, tag).
    // A lane owns 8 consecutive key tiles of the row (a head has at most 256), fetched by two 16-byte loads that
    // are both in flight before either is looked at.
    constexpr int kPerLane = 8;
    bool alive = true;
    for (int k = 0; k < K && alive; ++k) {
      const Item it = make_item<MT>(k, a);
      for (int r = it.c; r < a.M && alive; r += a.items_per_head) {
        const uint32_t* row = reinterpret_cast<const uint32_t*>(a.stats) + ((size_t)it.u * a.M + r) * a.tiles_pad;
        float v[kPerLane];
        uint32_t spins = 0;
        const bool has = 8 * lane < a.tiles_T;  // tiles_pad is a multiple of 8: the loads stay inside the row
        while (true) {
          uint32_t b[8] = {0xFF800000u, 0xFF800000u, 0xFF800000u, 0xFF800000u,
                           0xFF800000u, 0xFF800000u, 0xFF800000u, 0xFF800000u};  // -inf: neutral in the fold
          if (has)
            asm volatile(
                "ld.relaxed.gpu.global.v4.b32 {%0, %1, %2, %3}, [%8];\n\t"
                "ld.relaxed.gpu.global.v4.b32 {%4, %5, %6, %7}, [%8 + 16];"
                : "=r"(b[0]), "=r"(b[1]), "=r"(b[2]), "=r"(b[3]), "=r"(b[4]), "=r"(b[5]), "=r"(b[6]), "=r"(b[7])
                : "l"(row + 8 * lane)
                : "memory");
          bool all = true;
#pragma unroll
          for (int i = 0; i < kPerLane; ++i) {
            if (8 * lane + i < a.tiles_T) all = all && b[i] != kSentinel;
            else b[i] = 0xFF800000u;
            v[i] = __uint_as_float(b[i]);
          }
          if (__all_sync(0xffffffffu, all)) break;
          if (*abort_flag) {
            alive = false;
            break;
          }
          if (++spins > limit) {
            if (lane == 0) raise_abort(abort_flag, a.dev_status);
            alive = false;
            break;
          }
        }
        if (!alive) break;
        float mx = v[0];
#pragma unroll
        for (int i = 1; i < kPerLane; ++i) mx = fmaxf(mx, v[i]);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
        float sum = 0.f;
#pragma unroll
        for (int i = 0; i < kPerLane; ++i) sum += ex2(v[i] - mx);  // exp2(-inf) = 0; mx is finite: every row sees its own key
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
        if (lane == 0) {
          float2* out = reinterpret_cast<float2*>(a.lse) + (size_t)it.u * (128 * MT) + r;
          __stcg(out, make_float2(mx + log2f(sum), 1.f));
        }
      }
    }
  } else if (warp == kEpiWarps + 3) {
    // ---------------- log-sum-exp prefetch warp ----------------
    // Polls the (lse, tag) rows of the head of item k and puts -lse into shared memory for phase 2.
    for (int k = 0; k < K; ++k) {
      const Item it = make_item<MT>(k, a);
      const uint32_t slot = k & 1, par = (k >> 1) & 1;
      if (!mbar_wait(bar(P::kBarLseEmpty, slot), par ^ 1, abort_flag, a.dev_status, limit)) break;
      // a lane owns 4*MT consecutive rows: 2*MT 16-byte loads, all in flight before the first is looked at
      const float4* src = reinterpret_cast<const float4*>(a.lse) + (size_t)it.u * (64 * MT) + (2 * MT) * lane;
      float4 v[2 * MT];
      uint32_t spins = 0;
      bool got = false;
      while (true) {
        if constexpr (MT == 1)
          asm volatile(
              "ld.relaxed.gpu.global.v4.f32 {%0, %1, %2, %3}, [%8];\n\t"
              "ld.relaxed.gpu.global.v4.f32 {%4, %5, %6, %7}, [%8 + 16];"
              : "=f"(v[0].x), "=f"(v[0].y), "=f"(v[0].z), "=f"(v[0].w), "=f"(v[1].x), "=f"(v[1].y), "=f"(v[1].z),
                "=f"(v[1].w)
              : "l"(src)
              : "memory");
        else
          asm volatile(
              "ld.relaxed.gpu.global.v4.f32 {%0, %1, %2, %3}, [%16];\n\t"
              "ld.relaxed.gpu.global.v4.f32 {%4, %5, %6, %7}, [%16 + 16];\n\t"
              "ld.relaxed.gpu.global.v4.f32 {%8, %9, %10, %11}, [%16 + 32];\n\t"
              "ld.relaxed.gpu.global.v4.f32 {%12, %13, %14, %15}, [%16 + 48];"
              : "=f"(v[0].x), "=f"(v[0].y), "=f"(v[0].z), "=f"(v[0].w), "=f"(v[1].x), "=f"(v[1].y), "=f"(v[1].z),
                "=f"(v[1].w), "=f"(v[2].x), "=f"(v[2].y), "=f"(v[2].z), "=f"(v[2].w), "=f"(v[3].x), "=f"(v[3].y),
                "=f"(v[3].z), "=f"(v[3].w)
              : "l"(src)
              : "memory");
        bool mine = true;
#pragma unroll
        for (int jj = 0; jj < 2 * MT; ++jj) {
          const int row = (4 * MT) * lane + 2 * jj;
          if (row < a.M) mine = mine && v[jj].y != 0.f;
          if (row + 1 < a.M) mine = mine && v[jj].w != 0.f;
        }
        if (__all_sync(0xffffffffu, mine)) {
          got = true;
          break;
        }
        if (*abort_flag) break;
        if (++spins > limit) {
          if (lane == 0) raise_abort(abort_flag, a.dev_status);
          break;
        }
      }
      if (!got) break;
#pragma unroll
      for (int jj = 0; jj < 2 * MT; ++jj)
        *reinterpret_cast<float2*>(nlse_s + slot * 256 + (4 * MT) * lane + 2 * jj) = make_float2(-v[jj].x, -v[jj].z);
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(P::kBarLseFull, slot), 1);
    }
  } else {
    // ---------------- epilogue quads ----------------
    const int quad = warp >> 2, wq = warp & 3;
    const int qtid = threadIdx.x & 127;                           // TMEM lane of this thread in phase 1
    const uint32_t lane_addr = (uint32_t)(32 * wq) << 16;
    const int r = (MT == 2 ? 128 * quad : 0) + qtid;              // query row of this thread
    const int lim = r < a.M ? a.n + (r % a.w) : -1;                // last visible key; -1: padded row
    float m_slot0 = -INFINITY, m_slot1 = -INFINITY;                // reference of the exponentials parked in each slot
    bool alive = true;
    for (int step = 0; step <= K && alive; ++step) {
      if (step < K) {
        // ---- phase 1 of item `step`
        const Item it = make_item<MT>(step, a);
        const uint32_t slot = step & 1, par = (step >> 1) & 1, buf = 2 * slot + quad;
        const bool active = MT == 2 || quad < it.ntiles;
        const bool ok = mbar_wait(bar(P::kBarTFull, buf), par, abort_flag, a.dev_status, limit);
        if (ok && active) {
          tc_fence_after();
          const int tile = it.tile0 + (MT == 1 ? quad : 0);
          const int j0 = tile * kTileKeys;
          const uint32_t tcol = tmem_base + lane_addr + buf * 128;
          float m = -INFINITY, l = 0.f;
          if (j0 + kTileKeys > a.n) p1_tile<true>(tcol, j0, lim, a.scale_log2, m, l);   // reaches into the window / past T
          else p1_tile<false>(tcol, j0, lim, a.scale_log2, m, l);
          if (slot == 0) m_slot0 = m; else m_slot1 = m;
          if (r < a.M && it.index != a.drop_item)
            __stcg(a.stats + ((size_t)it.u * a.M + r) * a.tiles_pad + tile, l > 0.f ? m + log2f(l) : -INFINITY);
        }
      }
      if (step >= 1) {
        // ---- phase 2 of item `step - 1`
        const int k = step - 1;
        const Item it = make_item<MT>(k, a);
        const uint32_t slot = k & 1, par = (k >> 1) & 1, buf = 2 * slot + quad;
        const bool active = MT == 2 || quad < it.ntiles;
        const bool have_lse = mbar_wait(bar(P::kBarLseFull, slot), par, abort_flag, a.dev_status, limit);
        if (active) {
          // row factor of this thread's row; the phase-2 lanes fetch the four they need by shuffles (a warp's
          // 32 rows are the rows of its own 32 threads)
          const float mref = slot == 0 ? m_slot0 : m_slot1;
          const float cval = (have_lse && r < a.M) ? ex2(mref + nlse_s[slot * 256 + r]) : 0.f;
          const float c00 = __shfl_sync(0xffffffffu, cval, lane >> 2), c01 = __shfl_sync(0xffffffffu, cval, (lane >> 2) + 8);
          const float c10 = __shfl_sync(0xffffffffu, cval, (lane >> 2) + 16);
          const float c11 = __shfl_sync(0xffffffffu, cval, (lane >> 2) + 24);
          const uint32_t tq = tmem_base + lane_addr + buf * 128;
          const uint32_t hi16 = 16u << 16;
          uint64_t acc0[8], acc1[8];
          {
            float va[32], vb[32], vc[32], vd[32];
            tmem_ld_16x256b_x8(tq, va);
            tmem_ld_16x256b_x8(tq + hi16, vb);
            tmem_ld_16x256b_x8(tq + 64, vc);
            tmem_ld_16x256b_x8(tq + hi16 + 64, vd);
            tmem_ld_wait(va);
            tmem_ld_wait(vb);
            tmem_ld_wait(vc);
            tmem_ld_wait(vd);
            // the accumulator is free for the MMAs of the item after next
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(P::kBarTEmpty, buf), 1);
            p2_fma(acc0, va, c00, c01, true);
            p2_fma(acc0, vb, c10, c11, false);
            p2_fma(acc1, vc, c00, c01, true);
            p2_fma(acc1, vd, c10, c11, false);
          }
          const bool b4 = lane & 16, b3 = lane & 8, b2 = lane & 4;
          butterfly_round<4>(acc0, b4, 16);
          butterfly_round<4>(acc1, b4, 16);
          butterfly_round<2>(acc0, b3, 8);
          butterfly_round<2>(acc1, b3, 8);
          butterfly_round<1>(acc0, b2, 4);
          butterfly_round<1>(acc1, b2, 4);
          // lane t now holds the sums over the warp's 32 rows of columns 2t, 2t+1 (acc0[0]) and 64+2t, 64+2t+1 (acc1[0])
          // (the partial sums and the sampled flag alternate between two buffers: the barrier of the item in
          // between separates a reader of one item from the writers of the item after next)
          float* part_k = part_s + slot * 1024;
          uint64_t* pw = reinterpret_cast<uint64_t*>(part_k + warp * 128);
          pw[lane] = acc0[0];
          pw[32 + lane] = acc1[0];
          // Every thread reaches this barrier whatever its waits returned, and all threads that meet here take
          // the same decision to go on: one of them samples the abort flag for the others.
          const int grp = 2 * slot + (MT == 1 ? quad : 0);
          if ((MT == 1 ? qtid : (int)threadIdx.x) == 0) quad_abort[grp] = *abort_flag;
          if (MT == 1) bar_sync(1 + quad, 128); else bar_sync(3, 256);
          if (quad_abort[grp]) alive = false;
          const int tile = it.tile0 + (MT == 1 ? quad : 0);
          const int key = tile * kTileKeys + qtid;
          if (MT == 1) {
            const float* pq = part_k + quad * 512 + qtid;
            const float s = (pq[0] + pq[128]) + (pq[256] + pq[384]);
            if (key < a.n) a.raw[(size_t)it.u * a.n + key] = s;
          } else if (quad == 0) {
            const float* pq = part_k + qtid;
            const float s = ((pq[0] + pq[128]) + (pq[256] + pq[384])) + ((pq[512] + pq[640]) + (pq[768] + pq[896]));
            if (key < a.n) a.raw[(size_t)it.u * a.n + key] = s;
          }
        } else {
          // the item has no tile for this quad: only keep the accumulator's barriers in step
          __syncwarp();
          if (lane == 0) mbar_arrive(bar(P::kBarTEmpty, buf), 1);
        }
        __syncwarp();
        if (lane == 0 && have_lse) mbar_arrive(bar(P::kBarLseEmpty, slot), 1);
      }
    }
  }

  // ---------------- teardown ----------------
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    // give copies that may still be in flight time to land before the shared memory is released
    for (int i = 0; i < 64; ++i) __nanosleep(1000);
  }
  if (warp == kEpiWarps + 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

template <int MT>
cudaError_t launch_onepass(const CUtensorMap& qm, const CUtensorMap& km, OneArgs args, int grid, LaunchCtx& lc) {
  using P = OnePlan<MT>;
  const int smem = P::kTotal;
  auto kern = score_onepass_kernel<MT>;
  cudaError_t e;
  if ((e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem)) != cudaSuccess) return e;
  int per_sm = 0;
  if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, P::kThreads, smem)) != cudaSuccess) return e;
  if (per_sm < 1) return cudaErrorLaunchOutOfResources;
  void* params[] = {(void*)&qm, (void*)&km, (void*)&args};
  // cooperative launch: the CTAs of a head wait for one another, so all must be resident
  e = cudaLaunchCooperativeKernel((const void*)kern, dim3((unsigned)grid), dim3(P::kThreads), params, (size_t)smem,
                                  lc.st);
  lc.mark("score_onepass");
  return e != cudaSuccess ? e : cudaGetLastError();
}

int onepass_mt(const Dims& dm) { return dm.M > 128 ? 2 : 1; }
int onepass_tiles(const Dims& dm) { return (dm.T + kTileKeys - 1) / kTileKeys; }
int onepass_items_per_head(const Dims& dm) {
  const int per_item = onepass_mt(dm) == 1 ? 2 : 1;
  return (onepass_tiles(dm) + per_item - 1) / per_item;
}
int onepass_tiles_pad(const Dims& dm) { return (onepass_tiles(dm) + 7) & ~7; }

}  // namespace

// A head's work items must not outnumber the CTAs (each CTA parks at most two items in tensor memory and
// a head is complete only when all its items are parked).  128 CTAs is what a B200 offers with SMs to
// spare; the launcher re-checks against the device it runs on.
bool score_onepass_eligible(const Dims& dm) {
  return dm.dtype == LUKV_DTYPE_BF16 && dm.d == 128 && onepass_items_per_head(dm) <= kOnePassMaxItems;
}
size_t score_onepass_stats_bytes(const Dims& dm) {
  if (!score_onepass_eligible(dm)) return 0;
  return (size_t)dm.heads() * dm.M * onepass_tiles_pad(dm) * sizeof(float);
}

// Returns cudaErrorNotSupported (and launches nothing) when the device has fewer SMs than a head has items.
cudaError_t launch_score_onepass(const Dims& dm, const void* q, const void* k, const Workspace& ws, int32_t* dev_status,
                                 HeadRange hr, bool clear_flags, int spare_sms, LaunchCtx& lc) {
  int dev = 0, sms = 0;
  cudaError_t e;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
  if (spare_sms > 0 && sms > 8 * spare_sms) sms -= spare_sms;
  static const int cap = env_int("LUKV_SCORE_CTAS", 1, 1024, 0);  // tuning runs: fewer CTAs than SMs
  if (cap > 0 && cap < sms) sms = cap;
  OneArgs args;
  args.items_per_head = onepass_items_per_head(dm);
  if (args.items_per_head > sms) return cudaErrorNotSupported;
  CUtensorMap qm, km;
  if (!make_map(&qm, q, (uint64_t)dm.heads() * dm.M) || !make_map(&km, k, (uint64_t)dm.heads() * dm.T))
    return cudaErrorInvalidValue;
  args.stats = ws.stats;
  args.lse = reinterpret_cast<float*>(reinterpret_cast<char*>(ws.head_flags) + score_tc_lse_offset(dm));
  args.raw = ws.raw;
  args.dev_status = dev_status;
  args.M = dm.M;
  args.T = dm.T;
  args.w = dm.w;
  args.n = dm.n;
  args.head0 = hr.h0;
  args.nheads = hr.nh;
  args.tiles_T = onepass_tiles(dm);
  args.tiles_pad = onepass_tiles_pad(dm);
  args.scale_log2 = dm.scale_log2;
  score_test_hooks(&args.spin_limit, &args.drop_item);
  if (clear_flags) {
    // the (lse, tag) rows start at zero, the partials as all-ones bit patterns
    if ((e = cudaMemsetAsync(ws.head_flags, 0, score_tc_flag_bytes(dm), lc.st)) != cudaSuccess) return e;
    if ((e = cudaMemsetAsync(ws.stats, 0xFF, score_onepass_stats_bytes(dm), lc.st)) != cudaSuccess) return e;
  }
  const long long total_items = (long long)hr.nh * args.items_per_head;
  const int grid = (int)(total_items < sms ? total_items : sms);
  if (grid < args.items_per_head) return cudaErrorNotSupported;
  return dm.M > 128 ? launch_onepass<2>(qm, km, args, grid, lc) : launch_onepass<1>(qm, km, args, grid, lc);
}

}  // namespace lukv
