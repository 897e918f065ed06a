// Value norms of the oracle importance (Sec. 4.1, Eq. "oracle_importance"; App. E: L2 norm of the projected value),
//   vnorm[u][g][j] = || v[u][j] W_O^(g) ||_2 ,   u a KV head, g one of its G query heads, j a rankable position,
// on the tensor cores for bf16 inputs with d = 128.  Per (u, g) this is a dense contraction (n x d) * (d x D_model)
// followed by a sum of squares over the D_model output columns: 98 % of the flops of the importance computation.
//
// One persistent kernel, one CTA per SM, work items (u, g, chunk of 4096 positions).  For an item the CTA walks the
// projection in panels of 256 output columns and, per panel, the chunk's tiles of 128 positions:
//   warp 0      TMA producer: value tiles (128 positions x 128 channels, the layout of the key tiles of the scorer)
//   warp 1      allocates tensor memory; one lane issues the MMAs, D[position][column] = V tile * panel^T, N = 256
//   warps 2-5   epilogue: read the accumulator (a row per thread), add the squares to the row's running sum in
//               shared memory; after the last panel write the square roots
//   warps 6-9   panel writers: W_O^(g) is stored [d][D_model], the MMA wants each output column's 128 channels
//               contiguous, so the panel is transposed on its way into shared memory (8 loads of 4 columns -> 4 rows
//               of 8 channels, stored in the 128-byte-swizzled layout the MMA descriptor describes); a panel serves all
//               tiles of the chunk, and the next one is written while the current one is in use
// Every wait is bounded; the waits are between the warps of one CTA only.
#include "tc_ptx.cuh"

namespace lukv {
namespace {

constexpr int kVnRowTile = 128;                      // positions per MMA (M)
constexpr int kVnColTile = 256;                      // projection columns per MMA (N)
constexpr int kVnChunkTiles = 32;                    // row tiles per work item
constexpr int kVnChunkRows = kVnChunkTiles * kVnRowTile;
constexpr int kVnABytes = kVnRowTile * 128 * 2;      // one value tile: two halves of 64 channels
constexpr int kVnAHalf = kVnABytes / 2;
constexpr int kVnBBytes = kVnColTile * 128 * 2;      // one panel: two halves of 64 channels, 256 rows each
constexpr int kVnBHalf = kVnBBytes / 2;
constexpr int kVnThreads = 320;
constexpr int kVnSmem = 2 * kVnABytes + 2 * kVnBBytes + kVnChunkRows * 4 + 1024;

enum { kVnAFull = 0, kVnAEmpty = 2, kVnBFull = 4, kVnBEmpty = 6, kVnTFull = 8, kVnTEmpty = 10, kVnBars = 12 };

struct VnArgs {
  const __nv_bfloat16* w_o;  // [L][H*G][128][Dm]
  float* vnorm;              // [heads][G][n]
  int L, H, G, T, n, Dm;
  int chunks;                // row chunks per (u, g)
  long long items;           // heads * G * chunks
  uint32_t spin_limit;
};

// Writes the panel of output columns [m0, m0 + 256) of one projection slice w [128][Dm] into shared memory as 256
// rows (columns of W) of 128 channels, in two halves of 64 channels, rows of 128 bytes, 16-byte chunk c of row m at
// chunk position c ^ (m & 7).  Columns at or beyond Dm are zero.  128 threads.
__device__ __forceinline__ void vn_write_panel(unsigned char* panel, const __nv_bfloat16* w, int Dm, int m0, int t,
                                               bool vec) {
  if (vec) {
    // unit = (4 columns, 8 channels): 64 x 16 units, 8 per thread; lanes take consecutive column groups
    for (int unit = t; unit < 64 * 16; unit += 128) {
      const int mq = unit & 63, c8 = unit >> 6;
      const int m = m0 + 4 * mq;
      uint2 r[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        r[i] = make_uint2(0u, 0u);
        if (m < Dm) r[i] = __ldg(reinterpret_cast<const uint2*>(w + (size_t)(8 * c8 + i) * Dm + m));
      }
      const int half = c8 >> 3, c = c8 & 7;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        uint4 o;
        uint32_t* ow = reinterpret_cast<uint32_t*>(&o);
#pragma unroll
        for (int p = 0; p < 4; ++p) {
          const uint32_t a = k < 2 ? r[2 * p].x : r[2 * p].y, b = k < 2 ? r[2 * p + 1].x : r[2 * p + 1].y;
          ow[p] = __byte_perm(a, b, (k & 1) ? 0x7632 : 0x5410);
        }
        const int row = 4 * mq + k;
        *reinterpret_cast<uint4*>(panel + half * kVnBHalf + row * 128 + ((c ^ (row & 7)) << 4)) = o;
      }
    }
  } else {
    // any Dm and alignment: one column and 8 channels per unit
    for (int unit = t; unit < 256 * 16; unit += 128) {
      const int row = unit & 255, c8 = unit >> 8;
      const int m = m0 + row;
      uint4 o = make_uint4(0u, 0u, 0u, 0u);
      if (m < Dm) {
        uint32_t* ow = reinterpret_cast<uint32_t*>(&o);
        const unsigned short* ws = reinterpret_cast<const unsigned short*>(w);
#pragma unroll
        for (int p = 0; p < 4; ++p) {
          const uint32_t lo = __ldg(ws + (size_t)(8 * c8 + 2 * p) * Dm + m);
          const uint32_t hi = __ldg(ws + (size_t)(8 * c8 + 2 * p + 1) * Dm + m);
          ow[p] = lo | (hi << 16);
        }
      }
      const int half = c8 >> 3, c = c8 & 7;
      *reinterpret_cast<uint4*>(panel + half * kVnBHalf + row * 128 + ((c ^ (row & 7)) << 4)) = o;
    }
  }
}

struct VnItem {
  int u, g, row0, ntiles;
  const __nv_bfloat16* w;
};
__device__ __forceinline__ VnItem vn_item(const VnArgs& a, long long idx) {
  VnItem it;
  const int chunk = (int)(idx % a.chunks);
  const long long ug = idx / a.chunks;
  it.g = (int)(ug % a.G);
  it.u = (int)(ug / a.G);
  it.row0 = chunk * kVnChunkRows;
  it.ntiles = (min(kVnChunkRows, a.n - it.row0) + kVnRowTile - 1) / kVnRowTile;
  const int layer = (it.u / a.H) % a.L, h = it.u % a.H;
  it.w = a.w_o + ((size_t)layer * a.H * a.G + (size_t)h * a.G + it.g) * 128 * a.Dm;
  return it;
}

__global__ void __launch_bounds__(kVnThreads, 1)
    value_norm_tc_kernel(const __grid_constant__ CUtensorMap v_map, const VnArgs a) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  unsigned char* a_tiles = smem;                              // [2][kVnABytes]
  unsigned char* panels = smem + 2 * kVnABytes;               // [2][kVnBBytes]
  float* ssq = reinterpret_cast<float*>(panels + 2 * kVnBBytes);  // [kVnChunkRows] running sums of squares
  __shared__ __align__(8) uint64_t bars[kVnBars];
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_s;
  volatile int* abort_flag = &abort_s;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  auto bar = [&](int kind, int i) { return smem_u32(&bars[kind + i]); };

  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar(kVnAFull, i), 1);
      mbar_init(bar(kVnAEmpty, i), 1);
      mbar_init(bar(kVnBFull, i), 4);
      mbar_init(bar(kVnBEmpty, i), 1);
      mbar_init(bar(kVnTFull, i), 1);
      mbar_init(bar(kVnTEmpty, i), 4);
    }
    abort_s = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  for (int i = threadIdx.x; i < kVnChunkRows; i += kVnThreads) ssq[i] = 0.f;
  if (warp == 1) tmem_alloc(smem_u32(&tmem_slot), 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_slot;
  const int npanels = (a.Dm + kVnColTile - 1) / kVnColTile;

  if (warp == 0) {
    // ---------------- TMA producer: the value tiles, once per panel ----------------
    if (lane == 0) {
      uint32_t tt = 0;
      bool ok = true;
      for (long long idx = blockIdx.x; idx < a.items && ok; idx += gridDim.x) {
        const VnItem it = vn_item(a, idx);
        for (int cp = 0; cp < npanels && ok; ++cp)
          for (int rt = 0; rt < it.ntiles; ++rt, ++tt) {
            const uint32_t s = tt & 1, ph = (tt >> 1) & 1;
            if (!(ok = mbar_wait(bar(kVnAEmpty, s), ph ^ 1, abort_flag, nullptr, a.spin_limit))) break;
            mbar_expect_tx(bar(kVnAFull, s), kVnABytes);
            const uint32_t dst = smem_u32(a_tiles + s * kVnABytes);
            const int row = it.u * a.T + it.row0 + rt * kVnRowTile;  // rows past the head are never written back
            tma_load_2d(dst, &v_map, bar(kVnAFull, s), 0, row);
            tma_load_2d(dst + kVnAHalf, &v_map, bar(kVnAFull, s), 64, row);
          }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      constexpr uint32_t idesc = instr_desc_bf16(kVnRowTile, kVnColTile);
      uint32_t tt = 0, pc = 0;
      bool ok = true;
      for (long long idx = blockIdx.x; idx < a.items && ok; idx += gridDim.x) {
        const VnItem it = vn_item(a, idx);
        for (int cp = 0; cp < npanels && ok; ++cp, ++pc) {
          const uint32_t pb = pc & 1;
          if (!(ok = mbar_wait(bar(kVnBFull, pb), (pc >> 1) & 1, abort_flag, nullptr, a.spin_limit))) break;
          const uint32_t bp = smem_u32(panels + pb * kVnBBytes);
          for (int rt = 0; rt < it.ntiles; ++rt, ++tt) {
            const uint32_t s = tt & 1, ph = (tt >> 1) & 1;
            if (!(ok = mbar_wait(bar(kVnTEmpty, s), ph ^ 1, abort_flag, nullptr, a.spin_limit))) break;
            if (!(ok = mbar_wait(bar(kVnAFull, s), ph, abort_flag, nullptr, a.spin_limit))) break;
            tc_fence_after();
            const uint32_t at = smem_u32(a_tiles + s * kVnABytes);
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
              const int h = ks >> 2, sub = ks & 3;
              const uint64_t da = smem_desc_sw128(at + h * kVnAHalf) + (uint64_t)(sub * 2);
              const uint64_t db = smem_desc_sw128(bp + h * kVnBHalf) + (uint64_t)(sub * 2);
              umma_bf16(tmem_base + s * kVnColTile, da, db, idesc, ks > 0);
            }
            umma_commit(bar(kVnAEmpty, s));  // the value tile may be replaced once these MMAs have read it
            umma_commit(bar(kVnTFull, s));   // the accumulator is complete
          }
          if (ok) umma_commit(bar(kVnBEmpty, pb));  // the panel may be overwritten
        }
      }
    }
  } else if (warp < 6) {
    // ---------------- epilogue: a row per thread ----------------
    const int row = 32 * (warp & 3) + lane;  // a warp reads the TMEM lanes of its quadrant
    const uint32_t lane_addr = (uint32_t)(32 * (warp & 3)) << 16;
    uint32_t tt = 0;
    bool ok = true;
    for (long long idx = blockIdx.x; idx < a.items && ok; idx += gridDim.x) {
      const VnItem it = vn_item(a, idx);
      for (int cp = 0; cp < npanels && ok; ++cp)
        for (int rt = 0; rt < it.ntiles; ++rt, ++tt) {
          const uint32_t s = tt & 1, ph = (tt >> 1) & 1;
          if (!(ok = mbar_wait(bar(kVnTFull, s), ph, abort_flag, nullptr, a.spin_limit))) break;
          tc_fence_after();
          float ss0 = 0.f, ss1 = 0.f, ss2 = 0.f, ss3 = 0.f;
#pragma unroll 1
          for (int c0 = 0; c0 < kVnColTile; c0 += 32) {
            float v[32];
            tmem_ld32(tmem_base + lane_addr + s * kVnColTile + c0, v);
            tmem_ld_wait(v);
#pragma unroll
            for (int i = 0; i < 32; i += 4) {
              ss0 = fmaf(v[i], v[i], ss0);
              ss1 = fmaf(v[i + 1], v[i + 1], ss1);
              ss2 = fmaf(v[i + 2], v[i + 2], ss2);
              ss3 = fmaf(v[i + 3], v[i + 3], ss3);
            }
          }
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar(kVnTEmpty, s), 1);
          ssq[rt * kVnRowTile + row] += (ss0 + ss1) + (ss2 + ss3);  // only this thread touches this entry
        }
      if (!ok) break;
      float* out = a.vnorm + ((size_t)it.u * a.G + it.g) * a.n;
      for (int rt = 0; rt < it.ntiles; ++rt) {
        const int j = it.row0 + rt * kVnRowTile + row;
        if (j < a.n) out[j] = sqrtf(ssq[rt * kVnRowTile + row]);
        ssq[rt * kVnRowTile + row] = 0.f;
      }
    }
  } else {
    // ---------------- panel writers ----------------
    const int t = threadIdx.x - 6 * 32;
    const bool vec = (a.Dm & 3) == 0 && (reinterpret_cast<uintptr_t>(a.w_o) & 7) == 0;
    uint32_t pc = 0;
    bool ok = true;
    for (long long idx = blockIdx.x; idx < a.items && ok; idx += gridDim.x) {
      const VnItem it = vn_item(a, idx);
      for (int cp = 0; cp < npanels; ++cp, ++pc) {
        const uint32_t pb = pc & 1;
        if (!(ok = mbar_wait(bar(kVnBEmpty, pb), ((pc >> 1) & 1) ^ 1, abort_flag, nullptr, a.spin_limit))) break;
        vn_write_panel(panels + pb * kVnBBytes, it.w, a.Dm, cp * kVnColTile, t, vec);
        // the MMA reads shared memory through the asynchronous proxy: order these writes before it
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(kVnBFull, pb), 1);
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
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

}  // namespace

bool value_norm_tc_supported(const Dims& dm) {
  return dm.dtype == LUKV_DTYPE_BF16 && dm.d == 128 && dm.heads() * (int64_t)dm.T < ((int64_t)1 << 31);
}

cudaError_t launch_value_norm_tc(const Dims& dm, int d_model, const void* v, const void* w_o, float* vnorm,
                                 LaunchCtx& lc) {
  CUtensorMap vm;
  if (!make_map(&vm, v, (uint64_t)dm.heads() * dm.T)) return cudaErrorNotSupported;
  VnArgs a;
  a.w_o = static_cast<const __nv_bfloat16*>(w_o);
  a.vnorm = vnorm;
  a.L = dm.L, a.H = dm.H, a.G = dm.G, a.T = dm.T, a.n = dm.n, a.Dm = d_model;
  a.chunks = (dm.n + kVnChunkRows - 1) / kVnChunkRows;
  a.items = (long long)dm.heads() * dm.G * a.chunks;
  int drop = 0;
  score_test_hooks(&a.spin_limit, &drop);
  int dev = 0, sms = 0;
  cudaError_t e;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(value_norm_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kVnSmem)) != cudaSuccess)
    return e;
  const long long grid = a.items < sms ? a.items : sms;  // one CTA per SM: each owns the SM's tensor memory
  value_norm_tc_kernel<<<(unsigned)grid, kVnThreads, kVnSmem, lc.st>>>(vm, a);
  lc.mark("value_norm_tc");
  return cudaGetLastError();
}

}  // namespace lukv
