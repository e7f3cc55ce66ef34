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

// One block per 1024 survivors (256 threads x 4).  Reads the raw float32
// survivor values, writes codes (+ the block's scale) or halves, and block 0
// writes the payload header.
template <int BITS>
__global__ void __launch_bounds__(kCta)
k_quantize(const float* __restrict__ raw, unsigned long long k, unsigned long long n, Ctl* ctl,
           unsigned char* payload, PayloadLayout P) {
  __shared__ float s_max[kCta / 32];
  const unsigned long long j0 = (unsigned long long)blockIdx.x * NSML_QBLOCK + threadIdx.x * 4;

  if (blockIdx.x == 0 && threadIdx.x == 0) {
    nsml_payload_header h;
    h.magic = NSML_PAYLOAD_MAGIC;
    h.version = NSML_PAYLOAD_VERSION;
    h.n = n;
    h.k = k;
    h.bits = BITS;
    h.qblock = NSML_QBLOCK;
    h.nblocks = P.nblocks;
    h.idx_off = P.idx_off;
    h.val_off = P.val_off;
    h.scale_off = P.scale_off;
    *reinterpret_cast<nsml_payload_header*>(payload) = h;
    if (ctl->out_count != k && ctl->status == 0) set_status(&ctl->status, NSML_ERR_INTERNAL);
  }

  float v[4] = {0.f, 0.f, 0.f, 0.f};
  int cnt = 0;
  if (j0 + 4 <= k) {
    const float4 f = *reinterpret_cast<const float4*>(raw + j0);
    v[0] = f.x; v[1] = f.y; v[2] = f.z; v[3] = f.w;
    cnt = 4;
  } else if (j0 < k) {
    cnt = (int)(k - j0);
    for (int e = 0; e < cnt; ++e) v[e] = raw[j0 + e];
  }

  if (BITS == NSML_BITS_FP16) {
    uint16_t* out = reinterpret_cast<uint16_t*>(payload + P.val_off);
    if (cnt == 4) {
      uint2 w;
      w.x = (uint32_t)encode_f16(v[0]) | ((uint32_t)encode_f16(v[1]) << 16);
      w.y = (uint32_t)encode_f16(v[2]) | ((uint32_t)encode_f16(v[3]) << 16);
      *reinterpret_cast<uint2*>(out + j0) = w;
    } else {
      for (int e = 0; e < cnt; ++e) out[j0 + e] = encode_f16(v[e]);
    }
    return;
  }

  // block max-abs: warp shuffles, then one value per warp through shared memory
  float m = fmaxf(fmaxf(fabsf(v[0]), fabsf(v[1])), fmaxf(fabsf(v[2]), fabsf(v[3])));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
  if ((threadIdx.x & 31) == 0) s_max[threadIdx.x >> 5] = m;
  __syncthreads();
  m = s_max[0];
#pragma unroll
  for (int w = 1; w < kCta / 32; ++w) m = fmaxf(m, s_max[w]);
  const float scale = __fdiv_rn(m, 127.0f);
  if (threadIdx.x == 0) reinterpret_cast<float*>(payload + P.scale_off)[blockIdx.x] = scale;

  signed char* out = reinterpret_cast<signed char*>(payload + P.val_off);
  if (cnt == 4) {
    uint32_t w = 0;
#pragma unroll
    for (int e = 0; e < 4; ++e) w |= ((uint32_t)encode_i8(v[e], scale) & 0xFFu) << (8 * e);
    *reinterpret_cast<uint32_t*>(out + j0) = w;
  } else {
    for (int e = 0; e < cnt; ++e) out[j0 + e] = (signed char)encode_i8(v[e], scale);
  }
}

}  // namespace nsml
