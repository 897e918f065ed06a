// Stage (a) on the 5th-generation tensor cores (bf16, head_dim 128): one persistent kernel
// computes the un-pooled observation-window scores of every head.
//
// The window logits S = Q K^T of Eq. 1 (Sec. 3.1) come from tcgen05.mma with fp32
// accumulators in tensor memory; operands are staged in shared memory by TMA (128-byte
// swizzle, no multicast).  A row's softmax normaliser needs every key of the head before any
// probability is final, so each head is swept twice:
//   pass 1  D[query row][key]: a thread owns one query row in TMEM and folds its columns into
//           a (reference, sum-exp) pair; the partials of a work item go to global memory and
//           the CTA that delivers a head's last partial folds them into the row log-sum-exp
//   pass 2  D[key][query row] (operands swapped): a thread owns one key and adds
//           exp2(x - lse_row) over all rows in registers -> the un-pooled score of the key
// Both operand tiles are K-major, so the same shared-memory tiles serve as A or B.
//
// Work item = (head, run of item_tiles key tiles).  Items are dealt round-robin to a grid of
// at most one CTA per SM, launched cooperatively (all CTAs resident).  A CTA runs pass 1
// lag-1 items ahead of pass 2, so that the log-sum-exp of a head is normally complete before
// pass 2 needs it.  With small items the key tiles pass 2 re-reads are still in L2 (K crosses
// HBM once); the launcher prefers large items where there are enough of them, which re-read K
// from HBM but change jobs less often (the kernel is bound by the exp2 evaluation, not by HBM).
//
// Warp roles per CTA: 4*NQ epilogue warps in NQ quads (a warp may only read the TMEM lanes
// 32*(warp%4)..+31), then one warp each: TMA producer, MMA issuer 0 and TMEM owner, MMA issuer 1,
// helper (pass-1 partials -> global memory, head completion, -lse -> shared memory: it keeps every
// global-memory round trip off the epilogue warps).
// Every wait is bounded; a wait that runs out raises the CTA's abort flag and stores
// LUKV_ERR_TIMEOUT to the status word; the CTA then skips the remaining work and tears down
// normally.
#include "score_chunks.cuh"

namespace lukv {
namespace {


// ---- shared-memory layout ---------------------------------------------------------------------

template <int MT, int NQ>
struct Plan {
  static_assert(MT == 1 || NQ == 2, "two query-row blocks are split over exactly two quads");
  // An mbarrier wait only knows the parity of the phase it waits for, so the successive phases of a
  // barrier must be waited for by the same threads in order.  Accumulator buffer b = tile % kNumBufs is
  // read by quad tile % NQ and written by issuer tile % 2: both must be functions of b.
  // With three quads the buffers rotate over the quads, so "accumulator complete" has two barriers per
  // buffer, used alternately: a quad that runs ahead then still waits on a barrier whose previous
  // phase (eight tiles back) is long complete.
  static_assert(NQ == 2 || (MT == 1 && NQ == 3), "two quads, or three that take the tiles in turn");
  static constexpr int kEpiWarps = 4 * NQ;
  // + TMA producer, two MMA issuers, helper.  The count stays a multiple of 4 warps: the register
  // file is handed out as if the CTA were rounded up to one.
  static constexpr int kThreads = (kEpiWarps + 4) * 32;
  // Key-tile ring.  The count must be even: tile t uses stage t % kStages and is issued by issuer
  // t % 2, so with an even count every stage (its "full" barrier) has one waiting thread.  With an
  // odd count the two issuers would take turns on a stage, and the one that runs ahead could wait
  // for a phase two ahead of the barrier -- which a parity wait reports as complete while the
  // previous load of that stage is still in flight.
  static constexpr int kStages = MT == 1 ? 4 : 2;
  static_assert(kStages % 2 == 0, "a key stage must always be consumed by the same MMA issuer");
  static constexpr int kQSlots = 2;                    // query tiles of the job in the tensor pipe and the next one
  static constexpr int kQBytes = MT * kStageBytes;     // [half][MT*128 rows][128 B]
  static constexpr int kFinBufs = 1;                   // blocks of partials in flight while a head is folded
  static constexpr int kFinBytes = 16384;              // one block
  static constexpr int kFinParts = kFinBytes / (128 * MT * 4);  // items per block (one float per row and item)
  static constexpr int kKOff = kQSlots * kQBytes;
  static constexpr int kFinOff = kKOff + kStages * kStageBytes;
  static constexpr int kBarOff = kFinOff + kFinBufs * kFinBytes;
  static constexpr int kNumBufs = 4 / MT;              // accumulator buffers in TMEM
  static constexpr int kBufCols = 128 * MT;
  // barriers: full[kStages], empty[kStages], qfull[kQSlots], qempty[kQSlots], tfull[2][kNumBufs],
  // tempty[kNumBufs], pub_full[NQ], pub_empty[NQ], lse_full[kMaxLag], lse_empty[kMaxLag], fin[kFinBufs]
  static constexpr int kBarFull = 0, kBarEmpty = kStages, kBarQFull = 2 * kStages, kBarQEmpty = kBarQFull + kQSlots,
                       kBarTFull = kBarQEmpty + kQSlots, kBarTEmpty = kBarTFull + 2 * kNumBufs,
                       kBarPubFull = kBarTEmpty + kNumBufs, kBarPubEmpty = kBarPubFull + NQ,
                       kBarLseFull = kBarPubEmpty + NQ, kBarLseEmpty = kBarLseFull + kMaxLag,
                       kBarFin = kBarLseEmpty + kMaxLag, kNumBars = kBarFin + kFinBufs;
  static constexpr int kMiscOff = (kBarOff + kNumBars * 8 + 15) & ~15;  // tmem base, abort flag
  static constexpr int kPubOff = kMiscOff + 16;        // [NQ][128] (reference, sum-exp) handed to the publisher warp
  static constexpr int kLseOff = kPubOff + NQ * 128 * 8;  // [kMaxLag][256] -lse of the pass-2 jobs to come
  static_assert(kLseOff % 16 == 0, "lse rows are read with 16-byte loads");
  static constexpr int kTotal = kLseOff + kMaxLag * 256 * 4 + 1024;  // + slack for the 1024-byte alignment
  static_assert(kTotal <= 232448, "exceeds the shared memory of one CTA");
};

struct FusedArgs {
  float* stats;        // pass 1 partials: [heads][items_per_head][128*MT] log-sum-exp of the item's keys, exp2 domain
  float* lse;          // [heads][lse_rows] (row log-sum-exp in the exp2 domain, tag); zero at launch
  float* raw;          // pass 2 out: [heads][n]
  int* head_cnt;       // [heads] items whose partials were delivered (zero at launch)
  int32_t* dev_status;
  int M, T, w, n;
  int lse_rows;        // M rounded up to a multiple of 4
  int head0, nheads;   // heads [head0, head0+nheads) are scored by this launch
  int item_tiles, items_per_head, tiles_T, tiles_n;
  int adapt_items;     // host only: let the launcher pick a multiple of item_tiles
  int npad;            // pass 2: query rows rounded up to a multiple of 32 (MMA N and columns read)
  int lag;             // 2..kMaxLag: pass 1 of item k+lag-1 precedes pass 2 of item k
  int l2_hints;        // 1: pass-1 key loads ask L2 to keep the lines, pass-2 loads to drop them first
  float scale_log2;
  // sequences of different lengths in one launch (RAGGED kernels): seq_T[q] = context length of sequence q,
  // seq_item0[q] = number of its first work item; heads_per_seq heads each.  The uniform fields above then hold
  // the maxima (strides and capacities).  The tables travel by value in the launch arguments.
  int seq_T[kMaxRaggedSeqs], seq_item0[kMaxRaggedSeqs];
  int n_seq, heads_per_seq, total_items;
  int T_stride, n_stride;  // rows between consecutive heads in K and in the raw scores
  uint32_t spin_limit; // iterations a wait may take
  int drop_item;       // test hook: this work item's partials are stored but never counted in (-1: none)
};

struct Job {
  int u;       // head
  int c;       // item of the head
  int tile0;   // first key tile
  int ntiles;  // key tiles of this job (may be 0)
  int n;       // rankable positions of the head
  int iph;     // work items of the head
  bool p2;
};

template <bool RAGGED>
__device__ __forceinline__ Job make_job(int k, bool p2, const FusedArgs& a) {
  Job j;
  j.p2 = p2;
  const int item = (int)blockIdx.x + k * (int)gridDim.x;
  int tiles_T = a.tiles_T, tiles_n = a.tiles_n;
  if (!RAGGED) {
    j.n = a.n;
    j.iph = a.items_per_head;
    const int hu = item / a.items_per_head;
    j.c = item - hu * a.items_per_head;
    j.u = a.head0 + hu;
  } else {
    int lo = 0, hi = a.n_seq;  // the sequence whose items contain `item`
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (a.seq_item0[mid] <= item) lo = mid; else hi = mid;
    }
    const int2 sq = make_int2(a.seq_T[lo], a.seq_item0[lo]);
    j.n = sq.x - a.w;
    tiles_T = (sq.x + kTileKeys - 1) / kTileKeys;
    tiles_n = (j.n + kTileKeys - 1) / kTileKeys;
    j.iph = (tiles_T + a.item_tiles - 1) / a.item_tiles;
    const int local = item - sq.y, hu = local / j.iph;
    j.c = local - hu * j.iph;
    j.u = lo * a.heads_per_seq + hu;
  }
  j.tile0 = j.c * a.item_tiles;
  const int lim = p2 ? tiles_n : tiles_T;
  j.ntiles = max(0, min(a.item_tiles, lim - j.tile0));
  return j;
}

// Job `idx` of a CTA that owns K items: lag-1 pass-1 jobs first, then pass 1 of item k+lag-1
// alternating with pass 2 of item k, then the remaining pass-2 jobs.
template <bool RAGGED>
__device__ __forceinline__ Job decode_job(int idx, int K, const FusedArgs& a) {
  const int lead = min(a.lag - 1, K);
  if (idx < lead) return make_job<RAGGED>(idx, false, a);
  const int r = idx - lead, pairs = 2 * (K - lead);
  if (r < pairs) return (r & 1) ? make_job<RAGGED>(r >> 1, true, a) : make_job<RAGGED>(lead + (r >> 1), false, a);
  return make_job<RAGGED>(K - lead + (r - pairs), true, a);
}

template <int MT, int NQ, bool RAGGED>
__global__ void __launch_bounds__(Plan<MT, NQ>::kThreads, 1)
    score_fused_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap k_map,
                       const FusedArgs a) {
  using P = Plan<MT, NQ>;
  constexpr int kStages = P::kStages;
  constexpr int kNumBufs = P::kNumBufs;
  constexpr int kEpiWarps = P::kEpiWarps;
  constexpr int kRowsPad = 128 * MT;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sbase = smem_u32(smem);
  const uint32_t q_s = sbase;
  const uint32_t k_s = sbase + P::kKOff;
  const uint32_t bars = sbase + P::kBarOff;
  auto bar = [&](int first, int i) { return bars + 8u * (uint32_t)(first + i); };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + P::kMiscOff);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + P::kMiscOff + 4);
  float2* pub_s = reinterpret_cast<float2*>(smem + P::kPubOff);   // [NQ][128]
  float* nlse_s = reinterpret_cast<float*>(smem + P::kLseOff);    // [kMaxLag][256]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int total_items = a.total_items;
  const int K = (total_items - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;  // items of this CTA (>= 1)
  const int njobs = 2 * K;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(bar(P::kBarFull, s), 1);
      mbar_init(bar(P::kBarEmpty, s), 1);
    }
    for (int s = 0; s < P::kQSlots; ++s) {
      mbar_init(bar(P::kBarQFull, s), 1);
      mbar_init(bar(P::kBarQEmpty, s), 2);  // both MMA issuers
    }
    for (int b = 0; b < kNumBufs; ++b) {
      mbar_init(bar(P::kBarTFull, b), 1);
      mbar_init(bar(P::kBarTFull, kNumBufs + b), 1);
      mbar_init(bar(P::kBarTEmpty, b), MT == 2 ? 8 : 4);
    }
    for (int q = 0; q < NQ; ++q) {
      mbar_init(bar(P::kBarPubFull, q), 4);
      mbar_init(bar(P::kBarPubEmpty, q), 1);
    }
    for (int s = 0; s < kMaxLag; ++s) {
      mbar_init(bar(P::kBarLseFull, s), 1);
      mbar_init(bar(P::kBarLseEmpty, s), kEpiWarps);
    }
    for (int b = 0; b < P::kFinBufs; ++b) mbar_init(bar(P::kBarFin, b), 1);
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
      const uint64_t keep = l2_policy_evict_last(), drop = l2_policy_evict_first();
      uint32_t tt = 0, jq = 0;
      for (int idx = 0; idx < njobs; ++idx) {
        const Job j = decode_job<RAGGED>(idx, K, a);
        if (j.ntiles == 0) continue;
        const uint32_t slot = jq % P::kQSlots;
        if (!mbar_wait(bar(P::kBarQEmpty, slot), ((jq / P::kQSlots) & 1) ^ 1, abort_flag, a.dev_status, a.spin_limit)) break;
        mbar_expect_tx(bar(P::kBarQFull, slot), P::kQBytes);
        const uint32_t qd = q_s + slot * P::kQBytes;
        for (int h = 0; h < 2; ++h)
          for (int mt = 0; mt < MT; ++mt) {
            const uint32_t dst = qd + h * (MT * kHalfBytes) + mt * kHalfBytes;
            if (a.l2_hints) tma_load_2d_hint(dst, &q_map, bar(P::kBarQFull, slot), h * 64, j.u * a.M + mt * 128, keep);
            else tma_load_2d(dst, &q_map, bar(P::kBarQFull, slot), h * 64, j.u * a.M + mt * 128);
          }
        ++jq;
        bool ok = true;
        for (int t = 0; t < j.ntiles; ++t, ++tt) {
          const uint32_t s = tt % kStages, ph = (tt / kStages) & 1;
          if (!(ok = mbar_wait(bar(P::kBarEmpty, s), ph ^ 1, abort_flag, a.dev_status, a.spin_limit))) break;
          mbar_expect_tx(bar(P::kBarFull, s), kStageBytes);
          const int row = j.u * a.T_stride + (j.tile0 + t) * kTileKeys;
          const uint32_t dst = k_s + s * kStageBytes;
          if (a.l2_hints) {
            const uint64_t pol = j.p2 ? drop : keep;
            tma_load_2d_hint(dst, &k_map, bar(P::kBarFull, s), 0, row, pol);
            tma_load_2d_hint(dst + kHalfBytes, &k_map, bar(P::kBarFull, s), 64, row, pol);
          } else {
            tma_load_2d(dst, &k_map, bar(P::kBarFull, s), 0, row);
            tma_load_2d(dst + kHalfBytes, &k_map, bar(P::kBarFull, s), 64, row);
          }
        }
        if (!ok) break;
      }
    }
  } else if (warp == kEpiWarps + 1 || warp == kEpiWarps + 2) {
    // ---------------- MMA issuers ----------------
    // Two threads (in two warps) issue alternate key tiles.  A thread is held up by its waits and by
    // the tensor pipe's issue queue; with two of them one can wait while the other issues, so the
    // pipe does not idle between tiles.  Tiles that share an accumulator buffer or a key stage
    // (both have an even count) always belong to the same issuer, which keeps them in order.
    if (lane == 0) {
      const uint32_t me = warp == kEpiWarps + 1 ? 0u : 1u;
      uint32_t tt = 0, jq = 0;
      for (int idx = 0; idx < njobs; ++idx) {
        const Job j = decode_job<RAGGED>(idx, K, a);
        if (j.ntiles == 0) continue;
        const uint32_t slot = jq % P::kQSlots;
        const uint32_t qd = q_s + slot * P::kQBytes;
        bool ok = true, have_q = false;
        for (int t = 0; t < j.ntiles; ++t, ++tt) {
          if ((tt & 1) != me) continue;
          if (!have_q) {
            if (!(ok = mbar_wait(bar(P::kBarQFull, slot), (jq / P::kQSlots) & 1, abort_flag, a.dev_status, a.spin_limit))) break;
            have_q = true;
          }
          const uint32_t s = tt % kStages, ph = (tt / kStages) & 1;
          const uint32_t buf = tt % kNumBufs, use = tt / kNumBufs;
          if (!(ok = mbar_wait(bar(P::kBarTEmpty, buf), (use & 1) ^ 1, abort_flag, a.dev_status, a.spin_limit))) break;
          if (!(ok = mbar_wait(bar(P::kBarFull, s), ph, abort_flag, a.dev_status, a.spin_limit))) break;
          tc_fence_after();
          const uint32_t kt = k_s + s * kStageBytes;
          const uint32_t d_tmem = tmem_base + buf * P::kBufCols;
          if (!j.p2) {
            // D[q row][key]: A = Q (M-tile mt), B = K tile
            constexpr uint32_t idesc = instr_desc_bf16(128, kTileKeys);
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)
#pragma unroll
              for (int ks = 0; ks < 8; ++ks) {
                const int h = ks >> 2, sub = ks & 3;
                const uint64_t da = smem_desc_sw128(qd + h * (MT * kHalfBytes) + mt * kHalfBytes) + (uint64_t)(sub * 2);
                const uint64_t db = smem_desc_sw128(kt + h * kHalfBytes) + (uint64_t)(sub * 2);
                umma_bf16(d_tmem + mt * 128, da, db, idesc, ks > 0);
              }
          } else {
            // D[key][q row]: A = K tile, B = Q (npad rows)
            const uint32_t idesc = instr_desc_bf16(128, a.npad);
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
              const int h = ks >> 2, sub = ks & 3;
              const uint64_t da = smem_desc_sw128(kt + h * kHalfBytes) + (uint64_t)(sub * 2);
              const uint64_t db = smem_desc_sw128(qd + h * (MT * kHalfBytes)) + (uint64_t)(sub * 2);
              umma_bf16(d_tmem, da, db, idesc, ks > 0);
            }
          }
          umma_commit(bar(P::kBarEmpty, s));     // the stage may be refilled once these MMAs have read it
          umma_commit(bar(P::kBarTFull, buf + kNumBufs * (use & 1)));   // the accumulator is complete
        }
        if (!ok) break;
        umma_commit(bar(P::kBarQEmpty, slot));   // this issuer's share of the job no longer needs the query tiles
        ++jq;
      }
    }
  } else if (warp == kEpiWarps + 3) {
    // ---------------- helper: everything that needs a global-memory round trip ----------------
    // publish(k): merge the quads' pass-1 partials of item k, store them, count the item in
    //   (release).  The warp that counts a head's last item folds all its partials into the row
    //   log-sum-exp and stores it as (value, tag) pairs, zero at launch.
    // prefetch(k): poll those pairs for the head of item k (polling the data itself saves a flag
    //   round trip) and put -lse into shared memory for pass 2 of item k, which the quads reach
    //   several jobs after its pass 1.
    // Both are attempted in turn without blocking, so a head that completes late does not hold up
    // the publication of this CTA's next partials.
    uint32_t fin_uses[P::kFinBufs] = {};
    constexpr int kRowsLaneP = 4 * MT;
    int kp = 0, kf = 0;
    uint32_t p2c = 0, idle = 0;
    while ((kp < K || kf < K) && !*abort_flag) {
      bool progress = false;
      if (kp < K) {
        int ready = 1;
        if (lane == 0)
          for (int q = 0; q < NQ; ++q) ready &= (int)mbar_try_wait(bar(P::kBarPubFull, q), kp & 1);
        ready = __shfl_sync(0xffffffffu, ready, 0);
        if (ready) {
          const int k = kp;
          const bool ok = true;
          const Job j1 = make_job<RAGGED>(k, false, a);
          if (ok) {
            // one value per row: the log-sum-exp of the item's keys, m + log2(l); -inf for an empty partial
            float* dst = a.stats + ((size_t)j1.u * a.items_per_head + j1.c) * kRowsPad;
#pragma unroll
            for (int rr = 0; rr < kRowsPad; rr += 32) {
              float2 v = pub_s[rr + lane];
              if (MT == 1) {
                // the quads hold partials of the same 128 rows over different key tiles: merge them
#pragma unroll
                for (int q = 1; q < NQ; ++q) {
                  const float2 o = pub_s[q * 128 + rr + lane];
                  if (o.y > 0.f) {  // an empty partial is (-inf, 0)
                    const float mn = fmaxf(v.x, o.x);
                    v.y = v.y * ex2(v.x - mn) + o.y * ex2(o.x - mn);
                    v.x = mn;
                  }
                }
              }
              dst[rr + lane] = v.y > 0.f ? v.x + log2f(v.y) : -INFINITY;
            }
          }
          __syncwarp();
          if (lane == 0 && ok)
            for (int q = 0; q < NQ; ++q) mbar_arrive(bar(P::kBarPubEmpty, q), 1);
          // count the item in (release: the partials above; acquire: everybody else's)
          int last = 0;
          const bool dropped = (int)blockIdx.x + k * (int)gridDim.x == a.drop_item;
          if (lane == 0 && ok && !dropped && !*abort_flag)
            last = atom_add_acq_rel(a.head_cnt + j1.u, 1) == j1.iph - 1;
          last = __shfl_sync(0xffffffffu, last, 0);
          if (last) {
            // Fold the head's partials into lse = log2(sum_c 2^(v_c)).  The bulk-copy engine brings them
            // into shared memory (one round trip instead of one per load).  This warp competes with the
            // epilogue warps for issue slots and the head's consumers wait for the result, so the fold
            // is kept short: lane i owns rows 4i..4i+3 (one 16-byte load per item), terms are added
            // relative to the first item's value, and the exact two-sweep form (maximum first) is only
            // the fallback when that sum leaves a safe range.
            constexpr int kVecs = MT;  // float4 per lane and item
            const char* src = reinterpret_cast<const char*>(a.stats) + (size_t)j1.u * a.items_per_head * kRowsPad * 4;
            const int nblk = (j1.iph + P::kFinParts - 1) / P::kFinParts;
            auto request = [&](int blk) {  // lane 0
              const int parts = min(P::kFinParts, j1.iph - blk * P::kFinParts);
              const uint32_t bytes = (uint32_t)parts * kRowsPad * 4;
              mbar_expect_tx(bar(P::kBarFin, 0), bytes);
              bulk_load(sbase + P::kFinOff, src + (size_t)blk * P::kFinParts * kRowsPad * 4, bytes, bar(P::kBarFin, 0));
            };
            const float4* part = reinterpret_cast<const float4*>(smem + P::kFinOff);
            float ref[kVecs][4], sum[kVecs][4];
            bool fin_ok = true;
            for (int pass = 0; pass < 2 && fin_ok; ++pass) {  // pass 1 only if pass 0 left the safe range
              for (int blk = 0; blk < nblk && fin_ok; ++blk) {
                asm volatile("fence.proxy.async;" ::: "memory");
                __syncwarp();
                if (lane == 0) request(blk);
                fin_ok = mbar_wait(bar(P::kBarFin, 0), fin_uses[0] & 1, abort_flag, a.dev_status, a.spin_limit);
                ++fin_uses[0];
                if (!fin_ok) break;
                const int parts = min(P::kFinParts, j1.iph - blk * P::kFinParts);
                if (blk == 0) {
#pragma unroll
                  for (int vv = 0; vv < kVecs; ++vv) {
                    float4 r0 = part[vv * 32 + lane];
                    ref[vv][0] = r0.x, ref[vv][1] = r0.y, ref[vv][2] = r0.z, ref[vv][3] = r0.w;
                    sum[vv][0] = sum[vv][1] = sum[vv][2] = sum[vv][3] = 0.f;
                  }
                }
                if (pass == 1 && blk == 0) {
                  // the fallback needs the maximum of every row first; it is rare, so it simply reads the
                  // partials from global memory
                  const float4* g = reinterpret_cast<const float4*>(src);
                  for (int c = 0; c < j1.iph; ++c)
#pragma unroll
                    for (int vv = 0; vv < kVecs; ++vv) {
                      const float4 v = __ldcg(g + (size_t)c * (kRowsPad / 4) + vv * 32 + lane);
                      ref[vv][0] = fmaxf(ref[vv][0], v.x), ref[vv][1] = fmaxf(ref[vv][1], v.y);
                      ref[vv][2] = fmaxf(ref[vv][2], v.z), ref[vv][3] = fmaxf(ref[vv][3], v.w);
                    }
                }
                for (int c0 = 0; c0 < parts; c0 += 8)
#pragma unroll
                  for (int cc = 0; cc < 8; ++cc)
                    if (c0 + cc < parts) {
#pragma unroll
                      for (int vv = 0; vv < kVecs; ++vv) {
                        const float4 v = part[(c0 + cc) * (kRowsPad / 4) + vv * 32 + lane];
                        sum[vv][0] += ex2(v.x - ref[vv][0]);
                        sum[vv][1] += ex2(v.y - ref[vv][1]);
                        sum[vv][2] += ex2(v.z - ref[vv][2]);
                        sum[vv][3] += ex2(v.w - ref[vv][3]);
                      }
                    }
              }
              bool safe = true;
#pragma unroll
              for (int vv = 0; vv < kVecs; ++vv)
#pragma unroll
                for (int e = 0; e < 4; ++e)
                  if (4 * (vv * 32 + lane) + e < a.M) safe = safe && (sum[vv][e] >= 1e-30f) && (sum[vv][e] <= 1e30f);
              if (__all_sync(0xffffffffu, safe)) break;
            }
            float4* out = reinterpret_cast<float4*>(a.lse) + (size_t)j1.u * (a.lse_rows / 2);
#pragma unroll
            for (int vv = 0; vv < kVecs; ++vv) {
              const int row = 4 * (vv * 32 + lane);
              if (row < a.lse_rows && fin_ok) {
                __stcg(out + row / 2, make_float4(ref[vv][0] + log2f(sum[vv][0]), 1.f, ref[vv][1] + log2f(sum[vv][1]), 1.f));
                if (row + 2 < a.lse_rows)
                  __stcg(out + row / 2 + 1,
                         make_float4(ref[vv][2] + log2f(sum[vv][2]), 1.f, ref[vv][3] + log2f(sum[vv][3]), 1.f));
              }
            }
          }
          ++kp;
          progress = true;
        }
      }
      if (kf < kp) {
        const Job j2 = make_job<RAGGED>(kf, true, a);
        if (j2.ntiles == 0) {
          ++kf;
          progress = true;
        } else {
          const uint32_t slot = p2c % a.lag;
          int freeslot = 0;
          if (lane == 0) freeslot = (int)mbar_try_wait(bar(P::kBarLseEmpty, slot), ((p2c / a.lag) & 1) ^ 1);
          freeslot = __shfl_sync(0xffffffffu, freeslot, 0);
          if (freeslot) {
            const float2* src = reinterpret_cast<const float2*>(a.lse) + (size_t)j2.u * a.lse_rows;
            float2 v[kRowsLaneP];
            bool mine = true;
#pragma unroll
            for (int jj = 0; jj < kRowsLaneP; ++jj) {
              const int row = 32 * jj + lane;
              if (row < a.M) {
                v[jj] = ld_relaxed_f2(src + row);
                mine = mine && v[jj].y != 0.f;
              }
            }
            if (__all_sync(0xffffffffu, mine)) {
#pragma unroll
              for (int jj = 0; jj < 8; ++jj) {
                const int row = 32 * jj + lane;
                nlse_s[slot * 256 + row] = (jj < kRowsLaneP && row < a.M) ? -v[jj < kRowsLaneP ? jj : 0].x : -INFINITY;
              }
              __syncwarp();
              if (lane == 0) mbar_arrive(bar(P::kBarLseFull, slot), 1);
              ++p2c;
              ++kf;
              progress = true;
            }
          }
        }
      }
      if (progress) {
        idle = 0;
      } else {
        if (++idle > a.spin_limit) {
          if (lane == 0) raise_abort(abort_flag, a.dev_status);
          break;
        }
        if (idle > 8) __nanosleep(100);
      }
    }
  } else {
    // ---------------- epilogue quads ----------------
    const int quad = warp >> 2;
    const int qtid = threadIdx.x & 127;                          // TMEM lane of this thread
    const uint32_t lane_addr = (uint32_t)(32 * (warp & 3)) << 16;
    const uint64_t sc2 = pack2(a.scale_log2, a.scale_log2);
    uint32_t tt = 0, p1c = 0, p2c = 0;
    for (int idx = 0; idx < njobs; ++idx) {
      const Job j = decode_job<RAGGED>(idx, K, a);
      if (j.ntiles == 0) continue;
      if (!j.p2) {
        // ---- pass 1: (reference, sum-exp) of this thread's query row over the job's keys
        const int r = (MT == 2 ? 128 * quad : 0) + qtid;
        const int lim = r < a.M ? j.n + (r % a.w) : -1;           // last visible key; -1: padded row
        float m = -INFINITY, l = 0.f;
        for (int t = 0; t < j.ntiles; ++t, ++tt) {
          if (MT == 1 && (int)(tt % NQ) != quad) continue;
          const uint32_t buf = tt % kNumBufs, use = tt / kNumBufs;
          const bool ok = mbar_wait(bar(P::kBarTFull, buf + kNumBufs * (use & 1)), (use >> 1) & 1, abort_flag, a.dev_status, a.spin_limit);
          if (ok) {
            tc_fence_after();
            const int j0 = (j.tile0 + t) * kTileKeys;
            const bool masked = j0 + kTileKeys > j.n;             // tile reaches into the window / past T
            const uint32_t tcol = tmem_base + lane_addr + buf * P::kBufCols + (MT == 2 ? 128 * quad : 0);
            float va[32], vb[32];
            tmem_ld32(tcol, va);
#pragma unroll
            for (int c = 0; c < 4; c += 2) {
              tmem_ld_wait(va);
              tmem_ld32(tcol + 32 * (c + 1), vb);
              if (lim >= 0) {
                if (masked) p1_chunk<true>(va, j0 + 32 * c, lim, a.scale_log2, m, l);
                else p1_chunk<false>(va, j0 + 32 * c, lim, a.scale_log2, m, l);
              }
              tmem_ld_wait(vb);
              if (c + 2 < 4) tmem_ld32(tcol + 32 * (c + 2), va);
              if (lim >= 0) {
                if (masked) p1_chunk<true>(vb, j0 + 32 * (c + 1), lim, a.scale_log2, m, l);
                else p1_chunk<false>(vb, j0 + 32 * (c + 1), lim, a.scale_log2, m, l);
              }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(P::kBarTEmpty, buf), 1);
          }
        }
        // hand the partial to the publisher warp
        const bool ok = mbar_wait(bar(P::kBarPubEmpty, quad), (p1c & 1) ^ 1, abort_flag, a.dev_status, a.spin_limit);
        if (ok) pub_s[quad * 128 + qtid] = make_float2(m, l);
        __syncwarp();
        if (lane == 0 && ok) mbar_arrive(bar(P::kBarPubFull, quad), 1);
        ++p1c;
      } else {
        // ---- pass 2: this thread's key, summed over all query rows
        const uint32_t slot = p2c % a.lag;
        const bool have_lse = mbar_wait(bar(P::kBarLseFull, slot), (p2c / a.lag) & 1, abort_flag, a.dev_status, a.spin_limit);
        const float* nlse = nlse_s + slot * 256;
        for (int t = 0; t < j.ntiles; ++t, ++tt) {
          if ((int)(tt % NQ) != quad) continue;
          const uint32_t buf = tt % kNumBufs, use = tt / kNumBufs;
          const bool ok = mbar_wait(bar(P::kBarTFull, buf + kNumBufs * (use & 1)), (use >> 1) & 1, abort_flag, a.dev_status, a.spin_limit);
          if (ok) {
            tc_fence_after();
            const int key = (j.tile0 + t) * kTileKeys + qtid;
            const uint32_t tcol = tmem_base + lane_addr + buf * P::kBufCols;
            uint64_t acc0 = 0ull, acc1 = 0ull;
            float va[32], vb[32];
            tmem_ld32(tcol, va);
#pragma unroll 1
            for (int c0 = 0; c0 < a.npad; c0 += 64) {
              tmem_ld_wait(va);
              const bool two = c0 + 32 < a.npad;
              if (two) tmem_ld32(tcol + c0 + 32, vb);
              p2_chunk(va, nlse + c0, sc2, acc0, acc1);
              if (two) {
                tmem_ld_wait(vb);
                if (c0 + 64 < a.npad) tmem_ld32(tcol + c0 + 64, va);
                p2_chunk(vb, nlse + c0 + 32, sc2, acc0, acc1);
              }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(P::kBarTEmpty, buf), MT == 2 ? 2 : 1);
            if (key < j.n) a.raw[(size_t)j.u * a.n_stride + key] = sum4(acc0, acc1);
          }
        }
        __syncwarp();
        if (lane == 0 && have_lse) mbar_arrive(bar(P::kBarLseEmpty, slot), 1);
        ++p2c;
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

// ---- host side --------------------------------------------------------------------------------

template <int MT, int NQ, bool RAGGED = false>
cudaError_t launch_fused(const CUtensorMap& qm, const CUtensorMap& km, FusedArgs args, int spare_sms, LaunchCtx& lc,
                         const int32_t* seq_T_host = nullptr) {
  using P = Plan<MT, NQ>;
  const int smem = P::kTotal;
  auto kern = score_fused_kernel<MT, NQ, RAGGED>;
  cudaError_t e;
  if ((e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem)) != cudaSuccess) return e;
  int dev = 0, sms = 0, per_sm = 0;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
  if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, P::kThreads, smem)) != cudaSuccess) return e;
  if (per_sm < 1 || sms < 1) return cudaErrorLaunchOutOfResources;
  if (spare_sms > 0 && sms > 8 * spare_sms) sms -= spare_sms;
  // A CTA runs pass 1 of later items before pass 2 of the current one, so a head's items must
  // not outnumber the CTAs (else a CTA would wait for partials that it is due to produce itself).
  if (args.adapt_items) {
    // Larger work items mean fewer job changes and fewer partials to fold per head, but coarser dealing.
    // A CTA's critical path is its number of items times (tiles per item + about one tile's time of
    // per-item overhead); measured on 256 heads x 256 tiles and 148 CTAs: 0.89 ms with 8 tiles per item,
    // 0.84 with 16, 0.82 with 32, 0.81 with 64.  The price of large items is that pass 2 no longer finds all its key
    // tiles in L2; the kernel is bound by the exp2 unit, not by HBM, so re-reading part of K costs nothing.
    int best = args.item_tiles;
    double best_cost = 1e30;
    for (int mult = 1; mult <= 8; mult *= 2) {
      const int it = args.item_tiles * mult;
      const long long per_head = (args.tiles_T + it - 1) / it;
      const long long items = (long long)args.nheads * per_head;
      const long long ctas = items < sms ? items : sms;
      const double cost = (double)((items + ctas - 1) / ctas) * (it + 1.05);
      if (cost < best_cost * 0.995) {
        best_cost = cost;
        best = it;
      }
    }
    args.item_tiles = best;
  }
  while ((args.tiles_T + args.item_tiles - 1) / args.item_tiles > sms) ++args.item_tiles;
  args.items_per_head = (args.tiles_T + args.item_tiles - 1) / args.item_tiles;
  int total_items = args.nheads * args.items_per_head;
  if (RAGGED) {
    int base = 0;
    for (int q = 0; q < args.n_seq; ++q) {
      args.seq_T[q] = seq_T_host[q];
      args.seq_item0[q] = base;
      const int tiles = (seq_T_host[q] + kTileKeys - 1) / kTileKeys;
      base += args.heads_per_seq * ((tiles + args.item_tiles - 1) / args.item_tiles);
    }
    total_items = base;
  }
  args.total_items = total_items;
  const int grid = total_items < sms ? total_items : sms;  // one CTA per SM: each owns the SM's tensor memory
  void* params[] = {(void*)&qm, (void*)&km, (void*)&args};
  // cooperative launch: the CTAs of a head wait for one another, so all must be resident
  e = cudaLaunchCooperativeKernel((const void*)kern, dim3((unsigned)grid), dim3(P::kThreads), params, (size_t)smem,
                                  lc.st);
  lc.mark("score_fused");
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace

// Offset of the (lse, tag) rows inside the zero-initialised block that starts with the [heads] counters.
size_t score_tc_lse_offset(const Dims& dm) { return ((size_t)dm.heads() * sizeof(int) + 255) & ~(size_t)255; }

// Test hooks of the tensor-core scorers, read from the environment at every call: LUKV_TEST_SPIN_LIMIT shortens
// the limit of every device-side wait, LUKV_TEST_DROP_ITEM names one work item whose partial results never
// reach the other CTAs -- together they make a bounded wait run out without faulting anything.
void score_test_hooks(uint32_t* spin_limit, int* drop_item) {
  const char* lim = getenv("LUKV_TEST_SPIN_LIMIT");
  const char* drop = getenv("LUKV_TEST_DROP_ITEM");
  const long l = lim ? atol(lim) : 0, d = drop ? atol(drop) : -1;
  *spin_limit = (l >= 1 && l <= (1L << 30)) ? (uint32_t)l : kSpinLimit;
  *drop_item = (drop && d >= 0 && d <= (1L << 30)) ? (int)d : -1;
}

// Key tiles per work item (the smallest the scorer uses; it grows for very long contexts).
// LUKV_ITEM_TILES (1..64) overrides the default for tuning runs.
int score_item_tiles() {
  static const int v = env_int("LUKV_ITEM_TILES", 1, 64, 8);
  return v;
}
// Bytes of pass-1 partials the tensor-core scorer may write for these sizes.
size_t score_tc_stats_bytes(const Dims& dm) {
  const size_t tiles = ((size_t)dm.T + kTileKeys - 1) / kTileKeys;
  const size_t items = (tiles + score_item_tiles() - 1) / score_item_tiles();
  return (size_t)dm.heads() * items * 256 * 2 * sizeof(float);
}
// Bytes of the block that must be zero at launch: [heads] counters, then [heads][lse_rows][2] floats.
size_t score_tc_flag_bytes(const Dims& dm) {
  // the single-sweep kernel strides the rows of a head by 128 or 256, the two-sweep kernel by M rounded up to 4
  return score_tc_lse_offset(dm) + (size_t)dm.heads() * ((dm.M + 127) & ~127) * 2 * sizeof(float);
}

bool score_tc_supported(const Dims& dm) {
  return dm.dtype == LUKV_DTYPE_BF16 && dm.d == 128 && encode_fn() != nullptr;
}

cudaError_t launch_score_tc(const Dims& dm, const void* q, const void* k, const Workspace& ws, int32_t* dev_status,
                            HeadRange hr, bool clear_flags, int spare_sms, LaunchCtx& lc) {
  // The two-sweep kernel below is the default.  LUKV_SCORER=onesweep selects the single-sweep kernel where the
  // shape allows it (it parks a head's exponentials in tensor memory and is bound by the latency of the
  // log-sum-exp exchange between CTAs; at long contexts the two sweeps are faster).
  const char* which = getenv("LUKV_SCORER");
  if (which && which[0] == 'o' && !dm.seq_T && score_onepass_eligible(dm)) {
    const cudaError_t e1 = launch_score_onepass(dm, q, k, ws, dev_status, hr, clear_flags, spare_sms, lc);
    if (e1 != cudaErrorNotSupported) return e1;
  }
  CUtensorMap qm, km;
  if (!make_map(&qm, q, (uint64_t)dm.heads() * dm.M) || !make_map(&km, k, (uint64_t)dm.heads() * dm.T))
    return cudaErrorInvalidValue;
  FusedArgs args;
  args.stats = ws.stats;
  args.lse = reinterpret_cast<float*>(reinterpret_cast<char*>(ws.head_flags) + score_tc_lse_offset(dm));
  args.raw = ws.raw;
  args.head_cnt = ws.head_flags;
  args.dev_status = dev_status;
  args.M = dm.M;
  args.T = dm.T;
  args.w = dm.w;
  args.n = dm.n;
  args.T_stride = dm.T;
  args.n_stride = dm.n;
  args.n_seq = dm.S;
  args.heads_per_seq = dm.N;
  args.lse_rows = (dm.M + 3) & ~3;
  args.head0 = hr.h0;
  args.nheads = hr.nh;
  args.tiles_T = (dm.T + kTileKeys - 1) / kTileKeys;
  args.item_tiles = score_item_tiles();
  args.adapt_items = getenv("LUKV_ITEM_TILES") ? 0 : 1;
  args.tiles_n = (dm.n + kTileKeys - 1) / kTileKeys;
  args.items_per_head = 0;  // set by the launcher
  args.npad = (dm.M + 31) & ~31;
  static const int hints = env_int("LUKV_L2_HINTS", 0, 1, 1);
  args.l2_hints = hints;
  static const int lag = env_int("LUKV_LAG", 2, kMaxLag, 2);
  args.lag = lag;
  args.scale_log2 = dm.scale_log2;
  score_test_hooks(&args.spin_limit, &args.drop_item);
  // the per-head counters and the (value, tag) rows must start at zero; they are adjacent in the workspace
  if (clear_flags) {
    const cudaError_t e = cudaMemsetAsync(ws.head_flags, 0, score_tc_flag_bytes(dm), lc.st);
    if (e != cudaSuccess) return e;
  }
  if (dm.seq_T) {
    // sequences of different lengths: the whole call in one launch (no head ranges), work items dealt per sequence
    if (hr.h0 != 0 || hr.nh != (int)dm.heads() || dm.S > kMaxRaggedSeqs) return cudaErrorInvalidValue;
    return dm.M > 128 ? launch_fused<2, 2, true>(qm, km, args, spare_sms, lc, dm.seq_T)
                      : launch_fused<1, 2, true>(qm, km, args, spare_sms, lc, dm.seq_T);
  }
  if (dm.M > 128) return launch_fused<2, 2>(qm, km, args, spare_sms, lc);
  static const int quads = env_int("LUKV_QUADS", 2, 3, 2);
  if (quads == 3) return launch_fused<1, 3>(qm, km, args, spare_sms, lc);
  return launch_fused<1, 2>(qm, km, args, spare_sms, lc);
}

}  // namespace lukv
