// Oracle importance (Sec. 4.1, Eq. "oracle_importance"; App. E): for every cached position j of a KV head,
//   I_j = max over decode steps k of  sum_g A_{g,k,j} * || v_j W_O^(g) ||_2 ,
// A the attention weights (Eq. 1) of the G query heads of the KV head at decode step k, the softmax running over
// the T cached keys and, if decode keys are given, the keys of steps 1..k; each layer then divided by its total.
// An offline tool (it feeds the curve builder and the profile build), on the FP32 pipes in the tiling of the
// general-shape scorer: 64 x 64 dot products per shared-memory tile pair, a 4 x 4 register tile per thread.
//   value_norm_kernel   || v_j W_O^(g) ||_2 for every (head, g, rankable position)
//   imp_lse_kernel      row log-sum-exp of every (head, g, step), exp2 domain
//   imp_kernel          probabilities x value norms, summed over g inside a thread, maximum over the steps
//   imp_normalize_kernel  one CTA per (sequence, layer): fp64 total in a fixed order, then the division
#include <cstdlib>

#include "simt_tile.cuh"

namespace lukv {
namespace {

constexpr int kTile = 64;  // rows and keys (or projection columns) per shared-memory tile

// acc[a][kk] = <A row (rg + 16a), B row (kg + 16kk)> over D channels, both tiles fp32 with pitch D+4
template <int D>
__device__ __forceinline__ void tile_dots(const float* As, const float* Bs, int rg, int kg, float (&acc)[4][4]) {
  constexpr int kPitch = D + 4;
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) acc[a][kk] = 0.f;
#pragma unroll 4
  for (int c = 0; c < D; c += 4) {
    float4 bv[4];
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) bv[kk] = *reinterpret_cast<const float4*>(Bs + (kg + 16 * kk) * kPitch + c);
#pragma unroll
    for (int a = 0; a < 4; ++a) {
      const float4 av = *reinterpret_cast<const float4*>(As + (rg + 16 * a) * kPitch + c);
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) {
        acc[a][kk] = fmaf(av.x, bv[kk].x, acc[a][kk]);
        acc[a][kk] = fmaf(av.y, bv[kk].y, acc[a][kk]);
        acc[a][kk] = fmaf(av.z, bv[kk].z, acc[a][kk]);
        acc[a][kk] = fmaf(av.w, bv[kk].w, acc[a][kk]);
      }
    }
  }
}

struct ImpDims {
  int L, H, G, T, n, Kmax, Dm;
  float scale_log2;
};

// grid (heads * G, position tiles).  vnorm[(u*G + g)*n + j] = || v[u][j] W_O[layer][h*G+g] ||_2, j < n.
template <typename TIn, int D>
__global__ void __launch_bounds__(kSimtThreads) value_norm_kernel(const TIn* __restrict__ v, const TIn* __restrict__ w_o,
                                                                  float* __restrict__ vnorm, ImpDims dm) {
  constexpr int kPitch = D + 4;
  extern __shared__ __align__(16) float smem[];
  float* Vs = smem;                   // [64 positions][kPitch]
  float* Ws = smem + kTile * kPitch;  // [64 projection columns][kPitch]: a chunk of W_O, transposed
  const int u = blockIdx.x / dm.G, g = blockIdx.x % dm.G;
  const int layer = (u / dm.H) % dm.L, h = u % dm.H;
  const int j0 = blockIdx.y * kTile;
  const int tid = threadIdx.x, kg = tid & 15, rg = tid >> 4;
  const TIn* W = w_o + ((size_t)layer * dm.H * dm.G + (size_t)h * dm.G + g) * D * dm.Dm;
  load_rows_f32<TIn, D>(Vs, v + ((size_t)u * dm.T + j0) * D, kTile, min(kTile, dm.n - j0));
  float ss[4] = {0.f, 0.f, 0.f, 0.f};
  for (int m0 = 0; m0 < dm.Dm; m0 += kTile) {
    __syncthreads();  // the previous chunk is consumed (and Vs is complete on the first pass)
    for (int idx = tid; idx < D * kTile; idx += kSimtThreads) {
      const int c = idx / kTile, mm = idx % kTile;  // consecutive threads read consecutive projection columns
      Ws[mm * kPitch + c] = (m0 + mm < dm.Dm) ? to_f32(W[(size_t)c * dm.Dm + m0 + mm]) : 0.f;
    }
    __syncthreads();
    float acc[4][4];
    tile_dots<D>(Vs, Ws, rg, kg, acc);
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) ss[a] = fmaf(acc[a][kk], acc[a][kk], ss[a]);
  }
#pragma unroll
  for (int a = 0; a < 4; ++a) {
#pragma unroll
    for (int off = 1; off < 16; off <<= 1) ss[a] += __shfl_xor_sync(0xffffffffu, ss[a], off);
    const int j = j0 + rg + 16 * a;
    if (kg == 0 && j < dm.n) vnorm[((size_t)u * dm.G + g) * dm.n + j] = sqrtf(ss[a]);
  }
}

// Rows of a query tile: local row rg + 16a is (query head 4*gc + a, decode step k0 + rg), so a thread's four rows
// are four query heads at one step.  Rows beyond G or K_max are zero-filled.
template <typename TIn, int D>
__device__ __forceinline__ void load_query_tile(float* Qs, const TIn* q_dec, int u_q0, int gc, int k0, const ImpDims& dm) {
  constexpr int kPitch = D + 4;
  for (int a = 0; a < 4; ++a) {
    const int g = 4 * gc + a;
    const int valid = g < dm.G ? max(0, min(16, dm.Kmax - k0)) : 0;
    const size_t row0 = ((size_t)(u_q0 + min(g, dm.G - 1)) * dm.Kmax + min(k0, dm.Kmax - 1));
    load_rows_f32<TIn, D>(Qs + 16 * a * kPitch, q_dec + row0 * D, 16, valid);
  }
}

// grid (heads, step blocks of 16).  lse[(u*G + g)*Kmax + k] = log2 sum over visible keys of 2^(x*scale*log2 e).
template <typename TIn, int D>
__global__ void __launch_bounds__(kSimtThreads) imp_lse_kernel(const TIn* __restrict__ q_dec, const TIn* __restrict__ k,
                                                               const TIn* __restrict__ k_dec, float* __restrict__ lse,
                                                               ImpDims dm) {
  constexpr int kPitch = D + 4;
  extern __shared__ __align__(16) float smem[];
  float* Qs = smem;
  float* Ks = smem + kTile * kPitch;
  const int u = blockIdx.x, k0 = blockIdx.y * 16;
  const int tid = threadIdx.x, kg = tid & 15, rg = tid >> 4;
  const int u_q0 = u * dm.G;  // first query head of this KV head in the [S][L][H*G] order
  const int step = k0 + rg;
  for (int gc = 0; 4 * gc < dm.G; ++gc) {
    __syncthreads();
    load_query_tile<TIn, D>(Qs, q_dec, u_q0, gc, k0, dm);
    float row_m[4], row_l[4];
#pragma unroll
    for (int a = 0; a < 4; ++a) {
      row_m[a] = -INFINITY;
      row_l[a] = 0.f;
    }
    const int segs = k_dec ? 2 : 1;
    for (int seg = 0; seg < segs; ++seg) {
      const TIn* keys = seg == 0 ? k + (size_t)u * dm.T * D : k_dec + (size_t)u * dm.Kmax * D;
      const int count = seg == 0 ? dm.T : min(dm.Kmax, k0 + 16);     // decode keys beyond this block's steps are never visible
      const int lim = seg == 0 ? dm.T - 1 : step;                    // last visible key of this thread's rows in the segment
      for (int j0 = 0; j0 < count; j0 += kTile) {
        __syncthreads();
        load_rows_f32<TIn, D>(Ks, keys + (size_t)j0 * D, kTile, min(kTile, count - j0));
        __syncthreads();
        float acc[4][4];
        tile_dots<D>(Qs, Ks, rg, kg, acc);
#pragma unroll
        for (int a = 0; a < 4; ++a) {
          float x[4], tmax = -INFINITY;
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {
            const int j = j0 + kg + 16 * kk;
            x[kk] = (j <= lim && j < count) ? acc[a][kk] * dm.scale_log2 : -INFINITY;
            tmax = fmaxf(tmax, x[kk]);
          }
          if (tmax > -INFINITY) {
            const float mn = fmaxf(row_m[a], tmax);
            float l = row_l[a] * exp2f(row_m[a] - mn);
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) l += exp2f(x[kk] - mn);
            row_m[a] = mn;
            row_l[a] = l;
          }
        }
      }
    }
#pragma unroll
    for (int a = 0; a < 4; ++a) {
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
      const int g = 4 * gc + a;
      if (kg == 0 && g < dm.G && step < dm.Kmax) lse[((size_t)u * dm.G + g) * dm.Kmax + step] = m + log2f(l);
    }
  }
}

// grid (heads, key tiles of 64 rankable positions).
template <typename TIn, int D>
__global__ void __launch_bounds__(kSimtThreads) imp_kernel(const TIn* __restrict__ q_dec, const TIn* __restrict__ k,
                                                           const float* __restrict__ lse, const float* __restrict__ vnorm,
                                                           float* __restrict__ importance, ImpDims dm) {
  constexpr int kPitch = D + 4;
  extern __shared__ __align__(16) float smem[];
  float* Qs = smem;
  float* Ks = smem + kTile * kPitch;
  __shared__ float colmax[16][kTile];
  const int u = blockIdx.x, j0 = blockIdx.y * kTile;
  const int tid = threadIdx.x, kg = tid & 15, rg = tid >> 4;
  const int u_q0 = u * dm.G;
  load_rows_f32<TIn, D>(Ks, k + ((size_t)u * dm.T + j0) * D, kTile, min(kTile, dm.n - j0));
  float best[4] = {0.f, 0.f, 0.f, 0.f};  // importance is non-negative
  for (int k0 = 0; k0 < dm.Kmax; k0 += 16) {
    const int step = k0 + rg;
    float s[4] = {0.f, 0.f, 0.f, 0.f};   // sum over the query heads at this thread's step, for its four keys
    for (int gc = 0; 4 * gc < dm.G; ++gc) {
      __syncthreads();  // the previous query tile is consumed (and Ks is complete on the first pass)
      load_query_tile<TIn, D>(Qs, q_dec, u_q0, gc, k0, dm);
      __syncthreads();
      float acc[4][4];
      tile_dots<D>(Qs, Ks, rg, kg, acc);
#pragma unroll
      for (int a = 0; a < 4; ++a) {
        const int g = 4 * gc + a;
        if (g < dm.G && step < dm.Kmax) {
          const float row_lse = lse[((size_t)u * dm.G + g) * dm.Kmax + step];
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {
            const int j = j0 + kg + 16 * kk;
            if (j < dm.n)
              s[kk] = fmaf(exp2f(fmaf(acc[a][kk], dm.scale_log2, -row_lse)), vnorm[((size_t)u * dm.G + g) * dm.n + j], s[kk]);
          }
        }
      }
    }
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) best[kk] = fmaxf(best[kk], s[kk]);
  }
#pragma unroll
  for (int kk = 0; kk < 4; ++kk) colmax[rg][kg + 16 * kk] = best[kk];
  __syncthreads();
  if (tid < kTile && j0 + tid < dm.n) {
    float m = colmax[0][tid];
#pragma unroll
    for (int r = 1; r < 16; ++r) m = fmaxf(m, colmax[r][tid]);
    importance[(size_t)u * dm.n + j0 + tid] = m;
  }
}

// One CTA per (sequence, layer): the layer's H*n values are contiguous.  fp64 sum in a fixed order, then x / total.
__global__ void __launch_bounds__(1024) imp_normalize_kernel(float* __restrict__ importance, long long count) {
  __shared__ double part[32];
  __shared__ double total_s;
  float* base = importance + (size_t)blockIdx.x * count;
  double acc = 0.0;
  for (long long i = threadIdx.x; i < count; i += blockDim.x) acc += (double)base[i];
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double t = 0.0;
    for (int i = 0; i < (int)(blockDim.x >> 5); ++i) t += part[i];
    total_s = t;
  }
  __syncthreads();
  const double total = total_s;
  if (!(total > 0.0)) return;
  for (long long i = threadIdx.x; i < count; i += blockDim.x) base[i] = (float)((double)base[i] / total);
}

// LUKV_FORCE_SIMT=1 keeps the value norms on the FP32 pipes (for A/B checks; read at every call).
bool value_norm_force_simt() {
  const char* e = getenv("LUKV_FORCE_SIMT");
  return e && e[0] == '1';
}

template <typename TIn, int D>
cudaError_t launch_importance_t(const Dims& dm, ImpDims id, const void* q_dec, const void* k, const void* v,
                                const void* k_dec, const void* w_o, bool normalize, float* importance, float* vnorm,
                                float* lse, LaunchCtx& lc) {
  const size_t smem = (size_t)2 * kTile * (D + 4) * sizeof(float);
  cudaError_t e;
  auto kn = value_norm_kernel<TIn, D>;
  auto kl = imp_lse_kernel<TIn, D>;
  auto ki = imp_kernel<TIn, D>;
  if ((e = cudaFuncSetAttribute(kn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(kl, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(ki, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
  const unsigned heads = (unsigned)dm.heads();
  const unsigned pos_tiles = (unsigned)((dm.n + kTile - 1) / kTile);
  if (value_norm_tc_supported(dm) && !value_norm_force_simt()) {
    if ((e = launch_value_norm_tc(dm, id.Dm, v, w_o, vnorm, lc)) != cudaSuccess) return e;
  } else {
    kn<<<dim3(heads * id.G, pos_tiles), kSimtThreads, smem, lc.st>>>((const TIn*)v, (const TIn*)w_o, vnorm, id);
    lc.mark("value_norm");
  }
  kl<<<dim3(heads, (unsigned)((id.Kmax + 15) / 16)), kSimtThreads, smem, lc.st>>>((const TIn*)q_dec, (const TIn*)k,
                                                                                 (const TIn*)k_dec, lse, id);
  lc.mark("imp_lse");
  ki<<<dim3(heads, pos_tiles), kSimtThreads, smem, lc.st>>>((const TIn*)q_dec, (const TIn*)k, lse, vnorm, importance, id);
  lc.mark("importance");
  if (normalize) {
    imp_normalize_kernel<<<(unsigned)(dm.S * dm.L), 1024, 0, lc.st>>>(importance, (long long)dm.H * dm.n);
    lc.mark("imp_normalize");
  }
  return cudaGetLastError();
}

}  // namespace

size_t importance_workspace_bytes(const Dims& dm, int k_max) {
  const size_t a = ((size_t)dm.heads() * dm.G * dm.n * sizeof(float) + 255) & ~(size_t)255;
  const size_t b = ((size_t)dm.heads() * dm.G * k_max * sizeof(float) + 255) & ~(size_t)255;
  return a + b;
}

cudaError_t launch_importance(const Dims& dm, int k_max, int d_model, const void* q_dec, const void* k, const void* v,
                              const void* k_dec, const void* w_o, bool normalize, float* importance, void* ws,
                              LaunchCtx& lc) {
  ImpDims id;
  id.L = dm.L; id.H = dm.H; id.G = dm.G; id.T = dm.T; id.n = dm.n; id.Kmax = k_max; id.Dm = d_model;
  id.scale_log2 = dm.scale_log2;
  float* vnorm = static_cast<float*>(ws);
  float* lse = reinterpret_cast<float*>(static_cast<char*>(ws) +
                                        (((size_t)dm.heads() * dm.G * dm.n * sizeof(float) + 255) & ~(size_t)255));
  if (dm.dtype == LUKV_DTYPE_BF16) {
    if (dm.d == 128)
      return launch_importance_t<__nv_bfloat16, 128>(dm, id, q_dec, k, v, k_dec, w_o, normalize, importance, vnorm, lse, lc);
    return launch_importance_t<__nv_bfloat16, 64>(dm, id, q_dec, k, v, k_dec, w_o, normalize, importance, vnorm, lse, lc);
  }
  if (dm.d == 128)
    return launch_importance_t<float, 128>(dm, id, q_dec, k, v, k_dec, w_o, normalize, importance, vnorm, lse, lc);
  return launch_importance_t<float, 64>(dm, id, q_dec, k, v, k_dec, w_o, normalize, importance, vnorm, lse, lc);
}

}  // namespace lukv
