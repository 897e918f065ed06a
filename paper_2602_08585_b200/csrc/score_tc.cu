// Stage (a) on the 5th-generation tensor cores (bf16, head_dim 128): the window logits
// S = Q K^T of Eq. 1 (Sec. 3.1) are computed by tcgen05.mma with fp32 accumulators in
// tensor memory, operands staged in shared memory by TMA (128-byte swizzle, no multicast).
//
// Two sweeps over the keys of a head, each its own kernel:
//   sweep 1  D[query row][key]: every thread owns one query row in TMEM and folds its
//            columns into a running (max, sum-exp) -> per-chunk partials -> row log-sum-exp
//   sweep 2  D[key][query row] (operands swapped): every thread owns one key and adds
//            exp2(x - lse_row) over all rows in registers -> the un-pooled score of the key
// Both operand tiles are K-major, so the same shared-memory tiles serve as A or B.
//
// Warp roles per CTA (10 warps): 0-3 and 4-7 two epilogue quads (a warp may only read the
// TMEM lanes 32*(warp%4)..+31), 8 TMA producer, 9 MMA issuer and TMEM owner.
// Every wait is bounded; a wait that runs out raises the CTA's abort flag, stores
// LUKV_ERR_TIMEOUT to the status word and the CTA tears down normally.
#include <cuda.h>

#include "common.cuh"

namespace lukv {
namespace {

constexpr int kTileKeys = 128;                       // keys per shared-memory stage / per MMA M or N
constexpr int kTilesPerCta = 16;                     // key tiles per CTA
constexpr int kHalfBytes = kTileKeys * 128;          // one 64-channel half of a 128-row tile (SW128 atom rows)
constexpr int kStageBytes = 2 * kHalfBytes;          // 128 keys x 128 channels bf16
constexpr int kEpiWarps = 8;
constexpr int kThreads = (kEpiWarps + 2) * 32;
constexpr uint32_t kSpinLimit = 1u << 22;

// ---- PTX wrappers ------------------------------------------------------------------------

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: false when the CTA is aborting or the limit is reached (then it raises the abort).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* dev_status) {
  for (uint32_t i = 0; i < kSpinLimit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (i > 4096) __nanosleep(128);
  }
  *abort_flag = 1;
  if (dev_status) atomicExch(dev_status, (int32_t)LUKV_ERR_TIMEOUT);
  return false;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y)
      : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(cols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}

// D[tmem] (+)= A[smem] * B[smem]^T, bf16 inputs, fp32 accumulation; issued by one thread.
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, bool accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"((uint32_t)accumulate)
      : "memory");
}
// mbarrier arrives once every tcgen05.mma issued so far by this thread has completed
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// 32 lanes x 32 consecutive fp32 columns: thread i of the warp gets TMEM lane (base lane + i)
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
  uint32_t* r = reinterpret_cast<uint32_t*>(v);
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major tile stored as rows of 128 bytes with the
// 128-byte swizzle (8-row groups 1024 bytes apart), as written by TMA.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t saddr) {
  return (uint64_t)((saddr >> 4) & 0x3FFFu) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M x N tile.
__host__ __device__ constexpr uint32_t instr_desc_bf16(int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// ---- shared-memory layout ---------------------------------------------------------------------

template <int MT>
struct SmemPlan {
  static constexpr int kStages = MT == 2 ? 4 : 5;
  static constexpr int kQBytes = MT * kStageBytes;  // [half][MT*128 rows][128 B]
  static constexpr int kBarOff = kQBytes + kStages * kStageBytes;
  // barriers: full[kStages], empty[kStages], tfull[2], tempty[2], qfull
  static constexpr int kNumBars = 2 * kStages + 5;
  static constexpr int kMiscOff = (kBarOff + kNumBars * 8 + 15) & ~15;  // tmem base (4 B), abort flag (4 B)
  static constexpr int kLseOff = kMiscOff + 16;            // sweep 2: lse of up to 256 rows (read as float4: 16-byte aligned)
  static_assert(kLseOff % 16 == 0, "lse rows are read with 16-byte loads");
  static constexpr int kPartOff = kLseOff + 256 * 4;       // sweep 1, MT==1: (m,l) of the second quad
  static constexpr int kTotal = kPartOff + 128 * 8 + 1024;  // + slack for the 1024-byte alignment
};

struct ScoreTcArgs {
  float* stats;        // sweep 1 out: [heads][chunks][M][2]
  const float* lse;    // sweep 2 in : [heads][M]
  float* raw;          // sweep 2 out: [heads][n]
  int32_t* dev_status;
  int M, T, w, n, chunks;
  float scale_log2;
};

// One CTA: head u = blockIdx.x / chunks, key tiles [chunk*kTilesPerCta, ...).
template <int MT, bool SWEEP2>
__global__ void __launch_bounds__(kThreads, 1) score_tc_kernel(const __grid_constant__ CUtensorMap q_map,
                                                               const __grid_constant__ CUtensorMap k_map,
                                                               const ScoreTcArgs a) {
  using Plan = SmemPlan<MT>;
  constexpr int kStages = Plan::kStages;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sbase = smem_u32(smem);
  const uint32_t q_s = sbase;
  const uint32_t k_s = sbase + Plan::kQBytes;
  const uint32_t bars = sbase + Plan::kBarOff;
  auto bar_full = [&](int s) { return bars + 8u * s; };
  auto bar_empty = [&](int s) { return bars + 8u * (kStages + s); };
  auto bar_tfull = [&](int b) { return bars + 8u * (2 * kStages + b); };
  auto bar_tempty = [&](int b) { return bars + 8u * (2 * kStages + 2 + b); };
  const uint32_t bar_q = bars + 8u * (2 * kStages + 4);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + Plan::kMiscOff);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + Plan::kMiscOff + 4);
  float* lse_s = reinterpret_cast<float*>(smem + Plan::kLseOff);
  float2* part_s = reinterpret_cast<float2*>(smem + Plan::kPartOff);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int u = blockIdx.x / a.chunks, chunk = blockIdx.x % a.chunks;
  const int key_limit = SWEEP2 ? a.n : a.T;  // sweep 2 only needs the rankable keys
  const int tile0 = chunk * kTilesPerCta;
  const int tiles_total = (key_limit + kTileKeys - 1) / kTileKeys;
  const int ntiles = min(kTilesPerCta, tiles_total - tile0);
  const int npad = (a.M + 63) & ~63;  // sweep 2: query rows rounded up to the MMA N granularity used here

  // tiles per TMEM buffer use: sweep 1 with MT==2 fills one buffer (2 x 128 columns) per tile and both
  // quads read it; otherwise tile t goes to buffer t&1 and is read by quad t&1 alone.
  constexpr bool kBothQuads = (!SWEEP2 && MT == 2);
  constexpr uint32_t kBufCols = 256;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(bar_full(s), 1);
      mbar_init(bar_empty(s), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(bar_tfull(b), 1);
      mbar_init(bar_tempty(b), kBothQuads ? 8 : 4);
    }
    mbar_init(bar_q, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kEpiWarps + 1) tmem_alloc(smem_u32((const void*)tmem_slot), 512);
  if (SWEEP2) {
    for (int r = threadIdx.x; r < 256; r += kThreads)
      lse_s[r] = r < a.M ? a.lse[(size_t)u * a.M + r] : INFINITY;  // padded rows contribute exp2(-inf) = 0
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == kEpiWarps) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      mbar_expect_tx(bar_q, Plan::kQBytes);
      for (int h = 0; h < 2; ++h)
        for (int mt = 0; mt < MT; ++mt)
          tma_load_2d(q_s + h * (MT * kHalfBytes) + mt * kHalfBytes, &q_map, bar_q, h * 64, u * a.M + mt * 128);
      for (int t = 0; t < ntiles; ++t) {
        const int s = t % kStages;
        const uint32_t ph = (t / kStages) & 1;
        if (!mbar_wait(bar_empty(s), ph ^ 1, abort_flag, a.dev_status)) break;
        mbar_expect_tx(bar_full(s), kStageBytes);
        const int row = u * a.T + (tile0 + t) * kTileKeys;
        tma_load_2d(k_s + s * kStageBytes, &k_map, bar_full(s), 0, row);
        tma_load_2d(k_s + s * kStageBytes + kHalfBytes, &k_map, bar_full(s), 64, row);
      }
    }
  } else if (warp == kEpiWarps + 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      bool ok = mbar_wait(bar_q, 0, abort_flag, a.dev_status);
      for (int t = 0; ok && t < ntiles; ++t) {
        const int s = t % kStages;
        const uint32_t ph = (t / kStages) & 1;
        const int buf = kBothQuads ? (t & 1) : (t & 1);
        const uint32_t use = (uint32_t)(t >> 1);  // how often this buffer was used before
        if (!mbar_wait(bar_tempty(buf), (use & 1) ^ 1, abort_flag, a.dev_status)) break;
        if (!mbar_wait(bar_full(s), ph, abort_flag, a.dev_status)) break;
        tc_fence_after();
        const uint32_t kt = k_s + s * kStageBytes;
        const uint32_t d_tmem = tmem_base + buf * kBufCols;
        if (!SWEEP2) {
          // D[q row][key]: A = Q (M-tile mt), B = K tile
          constexpr uint32_t idesc = instr_desc_bf16(128, kTileKeys);
#pragma unroll
          for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
              const int h = ks >> 2, sub = ks & 3;
              const uint64_t da = smem_desc_sw128(q_s + h * (MT * kHalfBytes) + mt * kHalfBytes) + (uint64_t)(sub * 2);
              const uint64_t db = smem_desc_sw128(kt + h * kHalfBytes) + (uint64_t)(sub * 2);
              umma_bf16(d_tmem + mt * 128, da, db, idesc, ks > 0);
            }
        } else {
          // D[key][q row]: A = K tile, B = Q (npad rows)
          const uint32_t idesc = instr_desc_bf16(128, npad);
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {
            const int h = ks >> 2, sub = ks & 3;
            const uint64_t da = smem_desc_sw128(kt + h * kHalfBytes) + (uint64_t)(sub * 2);
            const uint64_t db = smem_desc_sw128(q_s + h * (MT * kHalfBytes)) + (uint64_t)(sub * 2);
            umma_bf16(d_tmem, da, db, idesc, ks > 0);
          }
        }
        umma_commit(bar_empty(s));     // the stage may be refilled once these MMAs have read it
        umma_commit(bar_tfull(buf));   // the accumulator is complete
      }
    }
  } else {
    // ---------------- epilogue quads ----------------
    const int quad = warp >> 2;
    const int lane_row = 32 * (warp & 3) + lane;                // TMEM lane of this thread
    const uint32_t lane_addr = (uint32_t)(32 * (warp & 3)) << 16;
    if (!SWEEP2) {
      const int r = (MT == 2 ? 128 * quad : 0) + lane_row;      // query row
      const int lim = r < a.M ? a.n + (r % a.w) : -1;           // last visible key
      float m = -INFINITY, l = 0.f;
      for (int t = 0; t < ntiles; ++t) {
        if (!kBothQuads && (t & 1) != quad) continue;
        const int buf = t & 1;
        const uint32_t use = (uint32_t)(t >> 1);
        if (!mbar_wait(bar_tfull(buf), use & 1, abort_flag, a.dev_status)) break;
        tc_fence_after();
        const int j0 = (tile0 + t) * kTileKeys;
        const bool masked = j0 + kTileKeys - 1 > a.n;            // tile reaches into the window / past T
        const uint32_t tcol = tmem_base + lane_addr + buf * kBufCols + (MT == 2 ? 128 * quad : 0);
#pragma unroll 1
        for (int c0 = 0; c0 < kTileKeys; c0 += 32) {
          float v[32];
          tmem_ld32(tcol + c0, v);
          tmem_ld_wait();
          // running max and exponent shift are kept in the scaled (exp2) domain; scale > 0
          float cmax = -INFINITY;
          if (masked) {
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              v[i] = (j0 + c0 + i <= lim) ? v[i] : -INFINITY;
              cmax = fmaxf(cmax, v[i]);
            }
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) cmax = fmaxf(cmax, v[i]);
          }
          if (lim < 0) cmax = -INFINITY;  // padded row
          if (cmax > -INFINITY) {
            const float mn = fmaxf(m, cmax * a.scale_log2);
            float acc = l * exp2f(m - mn);
#pragma unroll
            for (int i = 0; i < 32; ++i) acc += exp2f(fmaf(v[i], a.scale_log2, -mn));
            l = acc;
            m = mn;
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_tempty(buf));
      }
      // (m, l) of the row; with MT == 1 the two quads hold partials of the same rows
      if (MT == 1) {
        asm volatile("bar.sync 1, 256;" ::: "memory");
        if (quad == 1) part_s[lane_row] = make_float2(m, l);
        asm volatile("bar.sync 1, 256;" ::: "memory");
        if (quad == 0) {
          const float2 o = part_s[lane_row];
          const float mn = fmaxf(m, o.x);
          if (mn > -INFINITY) {
            l = l * exp2f(m - mn) + o.y * exp2f(o.x - mn);
            m = mn;
          }
        }
      }
      if ((MT == 2 || quad == 0) && r < a.M) {
        float* o = a.stats + (((size_t)u * a.chunks + chunk) * a.M + r) * 2;
        o[0] = m;
        o[1] = l;
      }
    } else {
      for (int t = 0; t < ntiles; ++t) {
        if ((t & 1) != quad) continue;
        const int buf = t & 1;
        const uint32_t use = (uint32_t)(t >> 1);
        if (!mbar_wait(bar_tfull(buf), use & 1, abort_flag, a.dev_status)) break;
        tc_fence_after();
        const int j = (tile0 + t) * kTileKeys + lane_row;        // key of this thread
        const uint32_t tcol = tmem_base + lane_addr + buf * kBufCols;
        float acc = 0.f;
#pragma unroll 1
        for (int c0 = 0; c0 < npad; c0 += 32) {
          float v[32];
          tmem_ld32(tcol + c0, v);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; i += 4) {
            const float4 ls = *reinterpret_cast<const float4*>(lse_s + c0 + i);
            acc += exp2f(fmaf(v[i], a.scale_log2, -ls.x));
            acc += exp2f(fmaf(v[i + 1], a.scale_log2, -ls.y));
            acc += exp2f(fmaf(v[i + 2], a.scale_log2, -ls.z));
            acc += exp2f(fmaf(v[i + 3], a.scale_log2, -ls.w));
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_tempty(buf));
        if (j < a.n) a.raw[(size_t)u * a.n + j] = acc;
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

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      p = nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

// 2-D bf16 tensor [rows][128] with boxes of 64 channels x 128 rows, 128-byte swizzle, zero fill.
bool make_map(CUtensorMap* map, const void* base, uint64_t rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {128, rows};
  const cuuint64_t strides[1] = {256};
  const cuuint32_t box[2] = {64, 128};
  const cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int MT>
cudaError_t launch_tc(const Dims& dm, const CUtensorMap& qm, const CUtensorMap& km, ScoreTcArgs args,
                      const Workspace& ws, LaunchCtx& lc) {
  const int smem = SmemPlan<MT>::kTotal;
  auto k1 = score_tc_kernel<MT, false>;
  auto k2 = score_tc_kernel<MT, true>;
  cudaError_t e;
  if ((e = cudaFuncSetAttribute(k1, cudaFuncAttributeMaxDynamicSharedMemorySize, smem)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(k2, cudaFuncAttributeMaxDynamicSharedMemorySize, smem)) != cudaSuccess) return e;
  const int keys_per_cta = kTileKeys * kTilesPerCta;
  const int chunks1 = (dm.T + keys_per_cta - 1) / keys_per_cta;
  const int chunks2 = (dm.n + keys_per_cta - 1) / keys_per_cta;
  args.chunks = chunks1;
  k1<<<(unsigned)(dm.heads() * chunks1), kThreads, smem, lc.st>>>(qm, km, args);
  lc.mark("score_tc_sweep1");
  if ((e = launch_lse(dm, ws.stats, ws.lse, chunks1, lc)) != cudaSuccess) return e;
  args.chunks = chunks2;
  k2<<<(unsigned)(dm.heads() * chunks2), kThreads, smem, lc.st>>>(qm, km, args);
  lc.mark("score_tc_sweep2");
  return cudaGetLastError();
}

}  // namespace

bool score_tc_supported(const Dims& dm) {
  return dm.dtype == LUKV_DTYPE_BF16 && dm.d == 128 && encode_fn() != nullptr;
}

cudaError_t launch_score_tc(const Dims& dm, const void* q, const void* k, const Workspace& ws, int32_t* dev_status,
                            LaunchCtx& lc) {
  CUtensorMap qm, km;
  if (!make_map(&qm, q, (uint64_t)dm.heads() * dm.M) || !make_map(&km, k, (uint64_t)dm.heads() * dm.T))
    return cudaErrorInvalidValue;
  ScoreTcArgs args;
  args.stats = ws.stats;
  args.lse = ws.lse;
  args.raw = ws.raw;
  args.dev_status = dev_status;
  args.M = dm.M;
  args.T = dm.T;
  args.w = dm.w;
  args.n = dm.n;
  args.chunks = 0;
  args.scale_log2 = dm.scale_log2;
  if (dm.M > 128) return launch_tc<2>(dm, qm, km, args, ws, lc);
  return launch_tc<1>(dm, qm, km, args, ws, lc);
}

}  // namespace lukv
