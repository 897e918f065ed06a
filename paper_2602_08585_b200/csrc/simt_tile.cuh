// Shared-memory tile loader of the FP32-pipe kernels (general-shape scorer, oracle importance).
#pragma once
#include "common.cuh"

namespace lukv {
namespace {

constexpr int kSimtThreads = 256;

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }

// Copy rows [row0, row0+rows) x D of a row-major global matrix into shared memory as fp32
// with a padded row pitch; rows at or beyond rows_valid are zero-filled.
template <typename TIn, int D>
__device__ __forceinline__ void load_rows_f32(float* dst, const TIn* src, int rows, int rows_valid) {
  constexpr int kPitch = D + 4;
  constexpr int kVec = 16 / sizeof(TIn);  // elements per 16-byte load
  constexpr int kVecPerRow = D / kVec;
  for (int idx = threadIdx.x; idx < rows * kVecPerRow; idx += kSimtThreads) {
    const int r = idx / kVecPerRow, cv = idx % kVecPerRow;
    float vals[kVec];
    if (r < rows_valid) {
      const uint4 raw = *reinterpret_cast<const uint4*>(src + (size_t)r * D + cv * kVec);
      const TIn* e = reinterpret_cast<const TIn*>(&raw);
#pragma unroll
      for (int t = 0; t < kVec; ++t) vals[t] = to_f32(e[t]);
    } else {
#pragma unroll
      for (int t = 0; t < kVec; ++t) vals[t] = 0.f;
    }
    float* o = dst + r * kPitch + cv * kVec;
#pragma unroll
    for (int t = 0; t < kVec; t += 4) *reinterpret_cast<float4*>(o + t) = make_float4(vals[t], vals[t + 1], vals[t + 2], vals[t + 3]);
  }
}

}  // namespace
}  // namespace lukv
