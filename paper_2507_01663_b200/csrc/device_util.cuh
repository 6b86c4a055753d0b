// Small device helpers shared by the kernels of the library.
#pragma once

#include <cuda_bf16.h>
#include <stdint.h>

namespace af {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// 2^x by the hardware approximation (about 2^-22 relative; denormal results flush to zero).
__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Two floats rounded to nearest-even bf16, packed low | high.
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}

// Sequence of a packed token: the largest j in [0, B) with cu[j] <= t  (cu non-decreasing,
// cu[0] = 0, t < cu[B]).  Bounded by log2 B steps whatever cu holds.
__device__ __forceinline__ int find_seq(const int32_t* __restrict__ cu, int B, int t) {
  int lo = 0, hi = B;
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (__ldg(cu + mid) <= t) lo = mid; else hi = mid;
  }
  return lo;
}

}  // namespace af
