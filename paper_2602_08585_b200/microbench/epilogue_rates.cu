// Micro-benchmark of the scorer's building blocks on one B200, timed with CUDA events and clock64:
//   - the tensor-core time of one 128x128x128 bf16 tile (tcgen05.mma, operands in shared memory)
//   - how many 128x128 accumulator tiles per SM the epilogue warps can turn from TMEM logits into sums,
//     with the kernel's own per-chunk functions (pass 1: row sums, pass 2: key sums), with exp2 only on the
//     special-function unit, and with exp2 only as the FMA-pipe polynomial; for one to three quads of four
//     warps, the two passes alone and side by side, with and without tensor-core work in the background.
// Nothing here synchronises warps with one another: these are the ceilings of the pieces, which the
// scorer's pipeline (accumulator hand-over, operand copies, the exchange between CTAs) cannot exceed.
#include <cstdio>
#include <cstdlib>

#include "score_chunks.cuh"
using namespace lukv;

namespace lukv_bench {

constexpr int kRoleKernel = 0, kRoleSfu = 1, kRolePoly = 2, kRoleMixed = 3, kRoleShfl = 4;  // mixed: SFU quads beside polynomial quads
constexpr int kMmaLimit = 1 << 22;

__device__ __forceinline__ void sfu_chunk(const float (&v)[32], uint64_t sc2, uint64_t nm2, uint64_t& acc0, uint64_t& acc1) {
#pragma unroll
  for (int i = 0; i < 32; i += 4) {
    acc0 = fadd2(acc0, ex2_pair(ffma2(pack2(v[i], v[i + 1]), sc2, nm2)));
    acc1 = fadd2(acc1, ex2_pair(ffma2(pack2(v[i + 2], v[i + 3]), sc2, nm2)));
  }
}
__device__ __forceinline__ void poly_chunk(const float (&v)[32], const float* nlse, uint64_t sc2, uint64_t& acc0,
                                           uint64_t& acc1) {
#pragma unroll
  for (int i = 0; i < 32; i += 4) {
    const ulonglong2 ls = *reinterpret_cast<const ulonglong2*>(nlse + i);
    acc0 = fadd2(acc0, ex2_poly_pair<false>(ffma2(pack2(v[i], v[i + 1]), sc2, ls.x)));
    acc1 = fadd2(acc1, ex2_poly_pair<false>(ffma2(pack2(v[i + 2], v[i + 3]), sc2, ls.y)));
  }
}

// Warps [0, 4*q1): pass-1 role; warps [4*q1, 4*(q1+q2)): pass-2 role; warp 15: background MMAs (mma_bg != 0).
// Each role processes `tiles` tiles per CTA, its quads taking them in turn out of TMEM buffers 0 and 1.
template <int ROLE>
__global__ void __launch_bounds__(512, 1) epilogue_rate(float* out, long long* clk, int tiles, int q1, int q2, int mma_bg) {
  extern __shared__ unsigned char dyn[];
  __shared__ uint32_t slot;
  __shared__ volatile int done_flag;
  __shared__ __align__(8) unsigned long long mbar;
  __shared__ __align__(16) float nlse[128];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x < 128) nlse[threadIdx.x] = -3.f - 0.01f * threadIdx.x;
  if (threadIdx.x == 0) {
    done_flag = 0;
    mbar_init(smem_u32(&mbar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) tmem_alloc(smem_u32(&slot), 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t base = slot;
  const uint32_t lane_addr = (uint32_t)(32 * (warp & 3)) << 16;
  if (warp < 4) {  // logits of ordinary size in buffers 0 and 1
    for (int c = 0; c < 8; ++c) {
      float r[32];
      for (int i = 0; i < 32; ++i) r[i] = -20.f + 0.05f * ((threadIdx.x * 7 + c * 32 + i) % 400);
      tmem_st32(base + lane_addr + c * 32, r);
    }
    tmem_st_wait();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const long long t0 = clock64();
  const uint64_t sc2 = pack2(0.1275f, 0.1275f), nm2 = pack2(-2.f, -2.f);
  uint64_t acc0 = 0ull, acc1 = 0ull;
  float m_run = -INFINITY, l_run = 0.f;
  const float4 mine4 = *reinterpret_cast<const float4*>(nlse + 4 * lane);
  const int quad = warp >> 2;
  if (quad < q1 + q2) {
    const bool first = quad < q1;
    const int nq = first ? q1 : q2;
    for (int t = first ? quad : quad - q1; t < tiles; t += nq) {
      const uint32_t tcol = base + lane_addr + (t & 1) * 128;
      float va[32], vb[32];
      tmem_ld32(tcol, va);
#pragma unroll
      for (int c = 0; c < 4; c += 2) {
        tmem_ld_wait(va);
        tmem_ld32(tcol + 32 * (c + 1), vb);
        if (first) {
          if (ROLE == kRoleKernel || ROLE == kRoleShfl) p1_chunk<false>(va, 0, 1 << 30, 0.1275f, m_run, l_run);
          else if (ROLE == kRoleSfu || ROLE == kRoleMixed) sfu_chunk(va, sc2, nm2, acc0, acc1);
          else poly_chunk(va, nlse + 32 * c, sc2, acc0, acc1);
        } else {
          if (ROLE == kRoleKernel) p2_chunk(va, nlse + 32 * c, sc2, acc0, acc1);
          else if (ROLE == kRoleShfl) p2_chunk_shfl(va, mine4, 32 * c, sc2, acc0, acc1);
          else if (ROLE == kRoleSfu) sfu_chunk(va, sc2, nm2, acc0, acc1);
          else poly_chunk(va, nlse + 32 * c, sc2, acc0, acc1);
        }
        tmem_ld_wait(vb);
        if (c + 2 < 4) tmem_ld32(tcol + 32 * (c + 2), va);
        if (first) {
          if (ROLE == kRoleKernel || ROLE == kRoleShfl) p1_chunk<false>(vb, 0, 1 << 30, 0.1275f, m_run, l_run);
          else if (ROLE == kRoleSfu || ROLE == kRoleMixed) sfu_chunk(vb, sc2, nm2, acc0, acc1);
          else poly_chunk(vb, nlse + 32 * (c + 1), sc2, acc0, acc1);
        } else {
          if (ROLE == kRoleKernel) p2_chunk(vb, nlse + 32 * (c + 1), sc2, acc0, acc1);
          else if (ROLE == kRoleShfl) p2_chunk_shfl(vb, mine4, 32 * (c + 1), sc2, acc0, acc1);
          else if (ROLE == kRoleSfu) sfu_chunk(vb, sc2, nm2, acc0, acc1);
          else poly_chunk(vb, nlse + 32 * (c + 1), sc2, acc0, acc1);
        }
      }
    }
  }
  long long mma_tiles = 0;
  if (warp == 15 && mma_bg && lane == 0) {
    // back-to-back 128x128x128 tiles into buffers 2 and 3 until the other warps are done (every loop bounded)
    const uint32_t sb = (smem_u32(dyn) + 1023) & ~1023u;
    constexpr uint32_t idesc = instr_desc_bf16(128, 128);
    uint32_t ph = 0;
    while (!done_flag && mma_tiles < kMmaLimit) {
      for (int ks = 0; ks < 8; ++ks) {
        const int h = ks >> 2, sub = ks & 3;
        const uint64_t da = smem_desc_sw128(sb + h * kHalfBytes) + (uint64_t)(sub * 2);
        const uint64_t db = smem_desc_sw128(sb + kStageBytes + h * kHalfBytes) + (uint64_t)(sub * 2);
        umma_bf16(base + (2 + (mma_tiles & 1)) * 128, da, db, idesc, ks > 0);
      }
      umma_commit(smem_u32(&mbar));
      for (int spin = 0; spin < (1 << 20) && !mbar_try_wait(smem_u32(&mbar), ph); ++spin) {}
      ph ^= 1;
      ++mma_tiles;
    }
  }
  const long long t1 = clock64();
  out[(size_t)blockIdx.x * 512 + threadIdx.x] = sum4(acc0, acc1) + m_run + l_run;
  if (lane == 0) clk[blockIdx.x * 32 + warp] = t1 - t0;
  if (warp == 15 && lane == 0) clk[blockIdx.x * 32 + 16] = mma_tiles;
  if (warp < 15) {
    asm volatile("bar.sync 1, 480;" ::: "memory");
    if (threadIdx.x == 0) done_flag = 1;
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(base, 512);
  }
}

// One thread issues `tiles` tiles back to back, each committed and waited for: tensor-core time per tile.
__global__ void __launch_bounds__(128, 1) mma_rate(long long* clk, int tiles) {
  extern __shared__ unsigned char dyn[];
  __shared__ uint32_t slot;
  __shared__ __align__(8) unsigned long long mbar[2];
  const int warp = threadIdx.x >> 5;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&mbar[0]), 1);
    mbar_init(smem_u32(&mbar[1]), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) tmem_alloc(smem_u32(&slot), 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t base = slot;
  if (threadIdx.x == 0) {
    const uint32_t sb = (smem_u32(dyn) + 1023) & ~1023u;
    constexpr uint32_t idesc = instr_desc_bf16(128, 128);
    const long long t0 = clock64();
    // two tiles in flight (buffers alternate), so the pipe never waits for the issuing thread
    for (int t = 0; t < tiles; ++t) {
      if (t >= 2)
        for (int spin = 0; spin < (1 << 20) && !mbar_try_wait(smem_u32(&mbar[t & 1]), ((t >> 1) - 1) & 1); ++spin) {}
      for (int ks = 0; ks < 8; ++ks) {
        const int h = ks >> 2, sub = ks & 3;
        const uint64_t da = smem_desc_sw128(sb + h * kHalfBytes) + (uint64_t)(sub * 2);
        const uint64_t db = smem_desc_sw128(sb + kStageBytes + h * kHalfBytes) + (uint64_t)(sub * 2);
        umma_bf16(base + (t & 3) * 128, da, db, idesc, ks > 0);
      }
      umma_commit(smem_u32(&mbar[t & 1]));
    }
    for (int b = 0; b < 2; ++b) {
      const int last = tiles - 1 - ((tiles - 1 - b) & 1);  // last tile committed to barrier b
      if (last >= 0)
        for (int spin = 0; spin < (1 << 22) && !mbar_try_wait(smem_u32(&mbar[b]), (last >> 1) & 1); ++spin) {}
    }
    clk[blockIdx.x] = clock64() - t0;
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(base, 512);
  }
}

template <int ROLE>
void run_case(const char* what, int q1, int q2, int mma_bg, float* out, long long* clk, int sms, int tiles) {
  const int smem = 70 * 1024;
  cudaFuncSetAttribute(epilogue_rate<ROLE>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  cudaEvent_t e0, e1;
  cudaEventCreate(&e0);
  cudaEventCreate(&e1);
  epilogue_rate<ROLE><<<sms, 512, smem>>>(out, clk, 64, q1, q2, mma_bg);  // warm-up
  cudaEventRecord(e0);
  epilogue_rate<ROLE><<<sms, 512, smem>>>(out, clk, tiles, q1, q2, mma_bg);
  cudaEventRecord(e1);
  if (cudaDeviceSynchronize() != cudaSuccess) {
    printf("CUDA error: %s\n", cudaGetErrorString(cudaGetLastError()));
    exit(1);
  }
  float ms;
  cudaEventElapsedTime(&ms, e0, e1);
  long long h[32];
  cudaMemcpy(h, clk, sizeof(h), cudaMemcpyDeviceToHost);  // CTA 0
  double c1 = 0, c2 = 0;
  for (int w = 0; w < 4 * q1; ++w) c1 += (double)h[w];
  for (int w = 4 * q1; w < 4 * (q1 + q2); ++w) c2 += (double)h[w];
  printf("| %-28s | %d | %d | %-3s | %8.3f | %6.0f | %6.0f |\n", what, q1, q2, mma_bg ? "yes" : "no", ms,
         q1 ? c1 / (4 * q1) / tiles : 0.0, q2 ? c2 / (4 * q2) / tiles : 0.0);
}

}  // namespace lukv_bench
using namespace lukv_bench;

int main() {
  int dev = 0, sms = 0, khz = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  cudaDeviceGetAttribute(&khz, cudaDevAttrClockRate, dev);
  float* out;
  long long* clk;
  cudaMalloc(&out, (size_t)sms * 512 * 4);
  cudaMalloc(&clk, (size_t)sms * 32 * 8);
  cudaMemset(clk, 0, (size_t)sms * 32 * 8);
  const int tiles = 4096;
  printf("%d SMs, max SM clock %d MHz; every case: %d tiles of 128x128 logits per role and SM\n", sms, khz / 1000, tiles);

  // tensor-core tile time
  {
    const int smem = 70 * 1024;
    cudaFuncSetAttribute(mma_rate, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    cudaEvent_t e0, e1;
    cudaEventCreate(&e0);
    cudaEventCreate(&e1);
    mma_rate<<<sms, 128, smem>>>(clk, 64);
    cudaEventRecord(e0);
    mma_rate<<<sms, 128, smem>>>(clk, tiles);
    cudaEventRecord(e1);
    if (cudaDeviceSynchronize() != cudaSuccess) {
      printf("CUDA error: %s\n", cudaGetErrorString(cudaGetLastError()));
      return 1;
    }
    float ms;
    cudaEventElapsedTime(&ms, e0, e1);
    long long c;
    cudaMemcpy(&c, clk, 8, cudaMemcpyDeviceToHost);
    printf("tcgen05.mma 128x128x128 bf16 tile: %.1f clocks per tile (%.3f ms for %d tiles on every SM: %.0f TFLOP/s)\n",
           (double)c / tiles, ms, tiles, 2.0 * 128 * 128 * 128 * tiles * sms / (ms * 1e-3) / 1e12);
  }

  printf("| epilogue code                | quads pass 1 | quads pass 2 | MMA | ms | clocks per tile, pass 1 | pass 2 |\n");
  printf("|---|---|---|---|---|---|---|\n");
  for (int q = 1; q <= 3; ++q) run_case<kRoleKernel>("kernel's chunk functions", q, 0, 0, out, clk, sms, tiles);
  for (int q = 1; q <= 3; ++q) run_case<kRoleKernel>("kernel's chunk functions", 0, q, 0, out, clk, sms, tiles);
  run_case<kRoleKernel>("kernel's chunk functions", 2, 0, 1, out, clk, sms, tiles);
  run_case<kRoleKernel>("kernel's chunk functions", 0, 2, 1, out, clk, sms, tiles);
  run_case<kRoleShfl>("pass 2, -lse by shuffles", 0, 2, 0, out, clk, sms, tiles);
  run_case<kRoleShfl>("pass 2, -lse by shuffles", 0, 2, 1, out, clk, sms, tiles);
  run_case<kRoleKernel>("kernel's chunk functions", 1, 1, 0, out, clk, sms, tiles);
  run_case<kRoleKernel>("kernel's chunk functions", 1, 1, 1, out, clk, sms, tiles);
  for (int q = 1; q <= 3; ++q) run_case<kRoleSfu>("exp2 on the SFU only", q, 0, 0, out, clk, sms, tiles);
  for (int q = 1; q <= 3; ++q) run_case<kRolePoly>("exp2 as polynomial only", 0, q, 0, out, clk, sms, tiles);
  // SFU quads (pass 1 column) beside polynomial quads (pass 2 column)
  run_case<kRoleMixed>("SFU quads | polynomial quads", 1, 1, 0, out, clk, sms, tiles);
  run_case<kRoleMixed>("SFU quads | polynomial quads", 1, 2, 0, out, clk, sms, tiles);
  run_case<kRoleMixed>("SFU quads | polynomial quads", 2, 2, 0, out, clk, sms, tiles);
  return 0;
}
