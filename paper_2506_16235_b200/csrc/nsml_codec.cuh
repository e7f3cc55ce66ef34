// Value codecs for the survivors (Alg. 2 Step 1 "quantize": float32 -> 16-bit
// float; plus a symmetric int8 codec with one max-abs scale per 1024 survivors,
// which the paper does not have).
#pragma once

#include "nsml_common.cuh"

namespace nsml {

// float32 -> binary16 bits, round to nearest even; a magnitude that would round
// to infinity (>= 65520) saturates to the largest finite half.
__device__ __forceinline__ uint16_t encode_f16(float v) {
  const float a = fabsf(v);
  if (a >= 65520.0f) return (uint16_t)((__float_as_uint(v) >> 16) & 0x8000u) | 0x7BFFu;
  return __half_as_ushort(__float2half_rn(v));
}

__device__ __forceinline__ float decode_f16(uint16_t h) { return __half2float(__ushort_as_half(h)); }

// code = clamp(rint(v / scale), +-127): one IEEE division, half to even.
__device__ __forceinline__ int encode_i8(float v, float scale) {
  if (scale == 0.0f) return 0;
  int c = __float2int_rn(__fdiv_rn(v, scale));
  return max(-127, min(127, c));
}

__device__ __forceinline__ float decode_i8(int code, float scale) { return __fmul_rn((float)code, scale); }

}  // namespace nsml
