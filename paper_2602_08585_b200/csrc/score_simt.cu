// Stage (a), general-shape scorer on the FP32 pipes (any dtype, d in {64,128}, up to 256
// score rows per head).  Two sweeps over the keys of a head:
//   sweep 1  logits of the window queries against a chunk of keys -> per-chunk row
//            (max, sum-exp) partials; a small kernel folds them into the row log-sum-exp
//   sweep 2  the same logits again -> probabilities -> column sums over the w window rows
//            and the G query heads (the "accumulated attention" of the proxy)
// followed by the 1-D max-pool.  Attention weights are Eq. 1 (Sec. 3.1) of the paper.
// Logits are kept in the exp2 domain: x2 = <q,k> * scale * log2(e).
#include "simt_tile.cuh"

namespace lukv {
namespace {

constexpr int kThreads = kSimtThreads;
constexpr int kKeyTile = 64;     // keys per shared-memory tile
constexpr int kChunkTiles = 16;  // tiles per CTA
constexpr int kChunk = kKeyTile * kChunkTiles;

// One CTA: all M rows of head u against keys [chunk*kChunk, +kChunk).
// Thread layout: kg = tid%16 owns keys {kg, kg+16, kg+32, kg+48} of a tile, rg = tid/16 owns
// rows {rg, rg+16, ...}.
template <typename TIn, int D, int RPT, bool SWEEP2>
__global__ void __launch_bounds__(kThreads) score_simt_kernel(const TIn* __restrict__ q, const TIn* __restrict__ k,
                                                              float* __restrict__ stats, const float* __restrict__ lse,
                                                              float* __restrict__ raw, int M, int T, int w, int chunks,
                                                              float scale_log2, SeqLens sl, int heads_per_seq) {
  constexpr int kPitch = D + 4;
  extern __shared__ __align__(16) float smem[];
  float* Qs = smem;                         // [16*RPT][kPitch]
  float* Ks = smem + 16 * RPT * kPitch;     // [kKeyTile][kPitch]
  __shared__ float colred[kThreads / 32][kKeyTile];

  const int u = blockIdx.x / chunks, chunk = blockIdx.x % chunks;
  // T is the row stride of the cache (the longest sequence); Tu the length of this head's sequence
  const int Tu = heads_per_seq > 0 ? sl.T[u / heads_per_seq] : T;
  const int n = Tu - w, n_stride = T - w;
  const int tid = threadIdx.x, kg = tid & 15, rg = tid >> 4;
  const TIn* qh = q + (size_t)u * M * D;
  const TIn* kh = k + (size_t)u * T * D;

  load_rows_f32<TIn, D>(Qs, qh, 16 * RPT, M);

  float row_m[RPT], row_l[RPT], row_lse[RPT];
  int row_lim[RPT];  // last visible key of the row
#pragma unroll
  for (int a = 0; a < RPT; ++a) {
    const int r = rg + 16 * a;
    row_m[a] = -INFINITY;
    row_l[a] = 0.f;
    row_lim[a] = r < M ? n + (r % w) : -1;
    row_lse[a] = 0.f;
    if (SWEEP2 && r < M) row_lse[a] = lse[(size_t)u * M + r];
  }

  const int key_begin = chunk * kChunk;
  const int key_end = min(Tu, key_begin + kChunk);
  for (int j0 = key_begin; j0 < key_end; j0 += kKeyTile) {
    __syncthreads();  // previous tile fully consumed (and Qs visible on the first pass)
    load_rows_f32<TIn, D>(Ks, kh + (size_t)j0 * D, kKeyTile, min(kKeyTile, Tu - j0));
    __syncthreads();

    float acc[RPT][4];
#pragma unroll
    for (int a = 0; a < RPT; ++a)
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) acc[a][kk] = 0.f;
#pragma unroll 4
    for (int c = 0; c < D; c += 4) {
      float4 kv[4];
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) kv[kk] = *reinterpret_cast<const float4*>(Ks + (kg + 16 * kk) * kPitch + c);
#pragma unroll
      for (int a = 0; a < RPT; ++a) {
        const float4 qv = *reinterpret_cast<const float4*>(Qs + (rg + 16 * a) * kPitch + c);
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
          acc[a][kk] = fmaf(qv.x, kv[kk].x, acc[a][kk]);
          acc[a][kk] = fmaf(qv.y, kv[kk].y, acc[a][kk]);
          acc[a][kk] = fmaf(qv.z, kv[kk].z, acc[a][kk]);
          acc[a][kk] = fmaf(qv.w, kv[kk].w, acc[a][kk]);
        }
      }
    }

    if (!SWEEP2) {
#pragma unroll
      for (int a = 0; a < RPT; ++a) {
        float x[4], tmax = -INFINITY;
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
          const int j = j0 + kg + 16 * kk;
          x[kk] = (j <= row_lim[a]) ? acc[a][kk] * scale_log2 : -INFINITY;
          tmax = fmaxf(tmax, x[kk]);
        }
        if (tmax > -INFINITY) {
          const float mn = fmaxf(row_m[a], tmax);
          float l = row_l[a] * exp2f(row_m[a] - mn);  // exp2f(-inf) = 0 on the first update
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) l += exp2f(x[kk] - mn);
          row_m[a] = mn;
          row_l[a] = l;
        }
      }
    } else {
      float cs[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int a = 0; a < RPT; ++a)
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
          const int j = j0 + kg + 16 * kk;
          if (j <= row_lim[a]) cs[kk] += exp2f(fmaf(acc[a][kk], scale_log2, -row_lse[a]));
        }
      // lanes l and l^16 hold the two row groups of this warp
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) cs[kk] += __shfl_xor_sync(0xffffffffu, cs[kk], 16);
      const int warp = tid >> 5;
      if ((tid & 16) == 0)
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) colred[warp][kg + 16 * kk] = cs[kk];
      __syncthreads();
      if (tid < kKeyTile) {
        float s = 0.f;
#pragma unroll
        for (int wv = 0; wv < kThreads / 32; ++wv) s += colred[wv][tid];
        const int j = j0 + tid;
        if (j < n) raw[(size_t)u * n_stride + j] = s;
      }
    }
  }

  if (!SWEEP2) {
    // fold the 16 key groups of each row (lanes differing in their low 4 bits)
#pragma unroll
    for (int a = 0; a < RPT; ++a) {
      float m = row_m[a], l = row_l[a];
#pragma unroll
      for (int off = 1; off < 16; off <<= 1) {
        const float mo = __shfl_xor_sync(0xffffffffu, m, off);
        const float lo = __shfl_xor_sync(0xffffffffu, l, off);
        const float mn = fmaxf(m, mo);
        if (mn > -INFINITY) {
          l = l * exp2f(m - mn) + lo * exp2f(mo - mn);
          m = mn;
        }
      }
      const int r = rg + 16 * a;
      if (kg == 0 && r < M) {
        float* o = stats + (((size_t)u * chunks + chunk) * M + r) * 2;
        o[0] = m;
        o[1] = l;
      }
    }
  }
}

// Fold the per-chunk partials of every row into lse2 = m + log2(l).
__global__ void score_lse_kernel(const float* __restrict__ stats, float* __restrict__ lse, int M, int chunks) {
  const int u = blockIdx.x;
  for (int r = threadIdx.x; r < M; r += blockDim.x) {
    float m = -INFINITY, l = 0.f;
    for (int c = 0; c < chunks; ++c) {
      const float* s = stats + (((size_t)u * chunks + c) * M + r) * 2;
      const float mo = s[0], lo = s[1];
      const float mn = fmaxf(m, mo);
      if (mn > -INFINITY) {
        l = l * exp2f(m - mn) + lo * exp2f(mo - mn);
        m = mn;
      }
    }
    lse[(size_t)u * M + r] = m + log2f(l);
  }
}

// n: row stride of the score arrays (the longest sequence); the head's own length comes from `sl` when the
// sequences differ (heads_per_seq > 0).
__global__ void max_pool_kernel(const float* __restrict__ raw, float* __restrict__ pooled, int n_stride, int half,
                                int tiles, int head0, SeqLens sl, int heads_per_seq, int w) {
  const int u = head0 + blockIdx.x / tiles;
  const int j = (blockIdx.x % tiles) * blockDim.x + threadIdx.x;
  const int n = heads_per_seq > 0 ? sl.T[u / heads_per_seq] - w : n_stride;
  if (j >= n) return;
  const float* r = raw + (size_t)u * n_stride;
  const int lo = max(0, j - half), hi = min(n - 1, j + half);
  float best = r[lo];
  for (int t = lo + 1; t <= hi; ++t) best = fmaxf(best, r[t]);
  pooled[(size_t)u * n_stride + j] = best;
}

// The same pooling, four outputs per thread with 16-byte accesses, for rows whose length is a multiple
// of four (then every row starts on a 16-byte boundary) and windows of at most nine positions: the
// outputs 4t..4t+3 need the inputs 4t-4..4t+7, three aligned vectors.  Positions outside [0,n) count
// as -inf (the window is clipped at the ends).
__global__ void max_pool4_kernel(const float4* __restrict__ raw, float4* __restrict__ pooled, int n4, int half,
                                 int tiles, int head0) {
  const int u = head0 + blockIdx.x / tiles;
  const int t = (blockIdx.x % tiles) * blockDim.x + threadIdx.x;
  if (t >= n4) return;
  const float4* r = raw + (size_t)u * n4;
  const float ninf = -INFINITY;
  const float4 a = t > 0 ? r[t - 1] : make_float4(ninf, ninf, ninf, ninf);
  const float4 b = r[t];
  const float4 c = t + 1 < n4 ? r[t + 1] : make_float4(ninf, ninf, ninf, ninf);
  const float x[12] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w, c.x, c.y, c.z, c.w};
  float y[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float best = x[4 + i];
#pragma unroll
    for (int d = 1; d <= 4; ++d)
      if (d <= half) best = fmaxf(best, fmaxf(x[4 + i - d], x[4 + i + d]));
    y[i] = best;
  }
  pooled[(size_t)u * n4 + t] = make_float4(y[0], y[1], y[2], y[3]);
}

template <typename TIn, int D, int RPT>
cudaError_t launch_sweeps(const Dims& dm, const void* q, const void* k, const Workspace& ws, LaunchCtx& lc) {
  cudaStream_t st = lc.st;
  const int chunks = score_chunks(dm);
  const size_t smem = (size_t)(16 * RPT + kKeyTile) * (D + 4) * sizeof(float);
  auto k1 = score_simt_kernel<TIn, D, RPT, false>;
  auto k2 = score_simt_kernel<TIn, D, RPT, true>;
  cudaError_t e;
  if ((e = cudaFuncSetAttribute(k1, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(k2, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
  const unsigned grid = (unsigned)(dm.heads() * chunks);
  SeqLens sl = {};
  const int heads_per_seq = dm.seq_T ? dm.N : 0;
  if (dm.seq_T)
    for (int q = 0; q < dm.S; ++q) sl.T[q] = dm.seq_T[q];
  k1<<<grid, kThreads, smem, st>>>((const TIn*)q, (const TIn*)k, ws.stats, nullptr, nullptr, dm.M, dm.T, dm.w, chunks,
                                   dm.scale_log2, sl, heads_per_seq);
  lc.mark("score_simt_sweep1");
  score_lse_kernel<<<(unsigned)dm.heads(), 256, 0, st>>>(ws.stats, ws.lse, dm.M, chunks);
  lc.mark("score_lse");
  k2<<<grid, kThreads, smem, st>>>((const TIn*)q, (const TIn*)k, nullptr, ws.lse, ws.raw, dm.M, dm.T, dm.w, chunks,
                                   dm.scale_log2, sl, heads_per_seq);
  lc.mark("score_simt_sweep2");
  return cudaGetLastError();
}

template <typename TIn, int D>
cudaError_t dispatch_rows(const Dims& dm, const void* q, const void* k, const Workspace& ws, LaunchCtx& lc) {
  const int rpt = (dm.M + 15) / 16;
  if (rpt <= 1) return launch_sweeps<TIn, D, 1>(dm, q, k, ws, lc);
  if (rpt <= 2) return launch_sweeps<TIn, D, 2>(dm, q, k, ws, lc);
  if (rpt <= 4) return launch_sweeps<TIn, D, 4>(dm, q, k, ws, lc);
  if (rpt <= 8) return launch_sweeps<TIn, D, 8>(dm, q, k, ws, lc);
  return launch_sweeps<TIn, D, 16>(dm, q, k, ws, lc);
}

}  // namespace

int score_chunks(const Dims& dm) { return (dm.T + kChunk - 1) / kChunk; }

cudaError_t launch_score_simt(const Dims& dm, const void* q, const void* k, const Workspace& ws, LaunchCtx& lc) {
  if (dm.dtype == LUKV_DTYPE_BF16) {
    if (dm.d == 64) return dispatch_rows<__nv_bfloat16, 64>(dm, q, k, ws, lc);
    return dispatch_rows<__nv_bfloat16, 128>(dm, q, k, ws, lc);
  }
  if (dm.d == 64) return dispatch_rows<float, 64>(dm, q, k, ws, lc);
  return dispatch_rows<float, 128>(dm, q, k, ws, lc);
}

cudaError_t launch_lse(const Dims& dm, const float* stats, float* lse, int chunks, LaunchCtx& lc) {
  score_lse_kernel<<<(unsigned)dm.heads(), 256, 0, lc.st>>>(stats, lse, dm.M, chunks);
  lc.mark("score_lse");
  return cudaGetLastError();
}

cudaError_t launch_pool(const Dims& dm, const float* raw, float* pooled, HeadRange hr, LaunchCtx& lc) {
  const int half = dm.kp / 2;
  const bool vec = !dm.seq_T && dm.n % 4 == 0 && half <= 4 && (reinterpret_cast<uintptr_t>(raw) & 15u) == 0 &&
                   (reinterpret_cast<uintptr_t>(pooled) & 15u) == 0;
  if (vec) {
    const int n4 = dm.n / 4, tiles = (n4 + 255) / 256;
    max_pool4_kernel<<<(unsigned)((int64_t)hr.nh * tiles), 256, 0, lc.st>>>(
        reinterpret_cast<const float4*>(raw), reinterpret_cast<float4*>(pooled), n4, half, tiles, hr.h0);
  } else {
    const int tiles = (dm.n + 255) / 256;
    SeqLens sl = {};
    if (dm.seq_T)
      for (int q = 0; q < dm.S; ++q) sl.T[q] = dm.seq_T[q];
    max_pool_kernel<<<(unsigned)((int64_t)hr.nh * tiles), 256, 0, lc.st>>>(raw, pooled, dm.n, half, tiles, hr.h0, sl,
                                                                           dm.seq_T ? dm.N : 0, dm.w);
  }
  lc.mark("max_pool");
  return cudaGetLastError();
}

}  // namespace lukv
