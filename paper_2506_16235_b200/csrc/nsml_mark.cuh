// Bucket -> candidate bitmap: the one full pass over the bucket (Alg. 2
// Steps 2-3: pruned gradients read as zero; every element whose magnitude
// reaches the sampled lower bound `lo` is marked as a candidate, everything
// else is dropped here, in one streaming read).
//
// The pass writes one bit per element (n / 8 bytes), a candidate count per
// group of kGroupElems elements and the candidates' histogram over kFineBins
// key bins above lo (bin width 2^shift, set by the sample kernel; the bins'
// counters are 128 bytes apart, because an L2 slice takes about one atomic per
// clock and the bins around the threshold are hot together).  It copies
// no values: the list stage reads the few marked elements again from the
// bucket.  Per 16-byte load a thread does four compares, three shuffles that
// assemble the 32-bit mask words of eight neighbouring lanes, and - for the one
// or two candidates per 128 elements - a fire-and-forget add to the global
// histogram, so the kernel stays at the rate of a plain read.
//
// Blocks walk the bucket block-cyclically in tiles of kStreamTile elements (the
// grid reads one moving window of memory); a thread keeps four 16-byte loads in
// flight.  There is no grid synchronisation, and no block synchronisation inside the loop.
#pragma once

#include "nsml_common.cuh"
#include "nsml_select.cuh"

namespace nsml {

// |v| >= t on floats equals key >= lo for finite v; written as !(|v| < t) so
// that NaN is kept too (the list stage reports non-finite candidates).
__device__ __forceinline__ unsigned int keep_flags(const uint32_t (&bits)[4], float t) {
  unsigned int f = 0;
#pragma unroll
  for (int e = 0; e < 4; ++e) f |= (unsigned)(!(fabsf(__uint_as_float(bits[e])) < t)) << e;
  return f;
}

// FEEDBACK: the bucket that is compressed is gradient + residual (Section 4.2 Step 3, local accumulation of
// the filtered gradients).  The residual is streamed beside the gradient, the sum (one float32 add per
// element) is written back over the residual and is what the candidates are taken from; the pruning mask
// zeroes a key, not the stored sum.
template <int DTYPE, bool FEEDBACK>
__global__ void __launch_bounds__(kCta)
k_mark(BucketSrc<DTYPE> src, float* __restrict__ residual, unsigned long long n, unsigned long long k, Ctl* ctl,
       uint32_t* __restrict__ bitmap, unsigned int* __restrict__ group_count, unsigned int* __restrict__ fine) {
  static_assert(kGroupElems % kStreamTile == 0, "a tile lies inside one group");
  // When every bin holds one key value (bfloat16 keys, massive ties) the candidates fall into a few dozen
  // bins, each of which would take tens of thousands of adds on one line of global memory: the block then
  // counts in shared memory and adds its non-empty bins to the global histogram once, at the end.
  __shared__ unsigned int s_fine[kFineBins];
  const bool privatise = ctl->exact != 0;
  if (privatise) {
    for (int b = threadIdx.x; b < kFineBins; b += kCta) s_fine[b] = 0;
    __syncthreads();
  }
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  // Zeros are never candidates; if they are needed (fewer than k non-zero keys) the candidates come out
  // short and the list stage falls back to the select over the bucket itself.
  const unsigned int lo = max(ctl->lo, 1u), shift = ctl->shift;  // (written by the sample kernel)
  const float t = __uint_as_float(lo);
  const unsigned long long tiles = (n + kStreamTile - 1) / kStreamTile;
  const unsigned long long nwords = ((n + kRoundElems - 1) / kRoundElems) * 4;  // whole rounds

  for (unsigned long long tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
    const unsigned long long base = tile * kStreamTile;
    uint32_t bits[kStreamLoads][4];
    const bool whole = base + kStreamTile <= n;
    if (whole) {
      if (!FEEDBACK) {
#pragma unroll
        for (int u = 0; u < kStreamLoads; ++u) src.load_full4(base + (unsigned long long)(u * kCta + threadIdx.x) * 4, bits[u]);
      } else {
        float4 r[kStreamLoads];
        unsigned int pm[kStreamLoads];
#pragma unroll
        for (int u = 0; u < kStreamLoads; ++u) {
          const unsigned long long i0 = base + (unsigned long long)(u * kCta + threadIdx.x) * 4;
          src.load_raw4(i0, bits[u]);
          r[u] = *reinterpret_cast<const float4*>(residual + i0);
          pm[u] = src.pruned4(i0);
        }
#pragma unroll
        for (int u = 0; u < kStreamLoads; ++u) {
          const unsigned long long i0 = base + (unsigned long long)(u * kCta + threadIdx.x) * 4;
          float4 acc;
          acc.x = __fadd_rn(__uint_as_float(bits[u][0]), r[u].x);
          acc.y = __fadd_rn(__uint_as_float(bits[u][1]), r[u].y);
          acc.z = __fadd_rn(__uint_as_float(bits[u][2]), r[u].z);
          acc.w = __fadd_rn(__uint_as_float(bits[u][3]), r[u].w);
          *reinterpret_cast<float4*>(residual + i0) = acc;
          bits[u][0] = (pm[u] & 1u) ? 0u : __float_as_uint(acc.x);
          bits[u][1] = (pm[u] & 2u) ? 0u : __float_as_uint(acc.y);
          bits[u][2] = (pm[u] & 4u) ? 0u : __float_as_uint(acc.z);
          bits[u][3] = (pm[u] & 8u) ? 0u : __float_as_uint(acc.w);
        }
      }
    } else {
      // the bucket's ragged last tile: plain loads, missing elements read as 0 and are never kept
#pragma unroll
      for (int u = 0; u < kStreamLoads; ++u) {
        const unsigned long long i0 = base + (unsigned long long)(u * kCta + threadIdx.x) * 4;
        if (!FEEDBACK) {
          src.load_vals4(i0, n, bits[u]);
        } else {
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const unsigned long long i = i0 + e;
            bits[u][e] = 0;
            if (i < n) {
              const float acc = __fadd_rn(__uint_as_float(src.raw1(i)), residual[i]);
              residual[i] = acc;
              bits[u][e] = src.pruned(i) ? 0u : __float_as_uint(acc);
            }
          }
        }
      }
    }
    unsigned int kept = 0, beyond = 0;  // beyond: candidates past the last fine bin's start (most of the sure survivors)
#pragma unroll
    for (int u = 0; u < kStreamLoads; ++u) {
      const unsigned int f = keep_flags(bits[u], t);
      kept += __popc(f);
      // the 4-bit flags of eight neighbouring lanes make one mask word (32 consecutive elements)
      unsigned int x = f << (4 * (lane & 7));
      x |= __shfl_xor_sync(0xFFFFFFFFu, x, 1);
      x |= __shfl_xor_sync(0xFFFFFFFFu, x, 2);
      x |= __shfl_xor_sync(0xFFFFFFFFu, x, 4);
      const unsigned long long word = base / 32 + (unsigned long long)u * (kCta / 8) + warp * 4 + (lane >> 3);
      if ((lane & 7) == 0 && (whole || word < nwords)) bitmap[word] = x;
      if (f != 0) {  // one or two candidates per 128 elements
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          if (f & (1u << e)) {
            const unsigned int bin = ((bits[u][e] & 0x7FFFFFFFu) - lo) >> shift;
            if (bin >= (unsigned int)(kFineBins - 1)) ++beyond;  // one hot counter: added once per warp and tile below
            else if (privatise) atomicAdd(&s_fine[bin], 1u);
            else atomicAdd(fine + bin * kFineStride, 1u);  // result unused: a reduction
          }
        }
      }
    }
    kept = __reduce_add_sync(0xFFFFFFFFu, kept);
    if (kept != 0) {  // warp-uniform
      beyond = __reduce_add_sync(0xFFFFFFFFu, beyond);
      if (lane == 0) {
        atomicAdd(group_count + base / kGroupElems, kept);
        if (beyond != 0) atomicAdd(fine + (kFineBins - 1) * kFineStride, beyond);
      }
    }
  }
  if (privatise) {
    __syncthreads();
    for (int b = threadIdx.x; b < kFineBins - 1; b += kCta) {
      const unsigned int c = s_fine[b];
      if (c != 0) atomicAdd(fine + b * kFineStride, c);
    }
  }

  // The block that finishes last resolves the fine bin that holds the k-th largest key, once for everybody:
  // the list stage starts from it.  (Every thread's adds are ordered before its block's ticket.)
  __shared__ unsigned int s_tot[kCta / 32], s_out[2], s_last;
  __shared__ unsigned long long s_sum[kCta / 32];
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) s_last = atomicAdd(&ctl->mark_done, 1u) == gridDim.x - 1;
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  constexpr int PER = kFineBins / kCta;
  unsigned int own[PER];
  unsigned long long mine = 0;
#pragma unroll
  for (int b = 0; b < PER; ++b) {
    own[b] = __ldcg(fine + (size_t)(threadIdx.x * PER + b) * kFineStride);
    mine += own[b];
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mine += __shfl_xor_sync(0xFFFFFFFFu, mine, o);
  if (lane == 0) s_sum[warp] = mine;
  __syncthreads();
  unsigned long long total = 0;
#pragma unroll
  for (int w = 0; w < kCta / 32; ++w) total += s_sum[w];
  if (total < k) {  // fewer candidates than survivors: the select runs over the bucket itself
    if (threadIdx.x == 0) ctl->fallback = 1u;
    return;
  }
  find_digit_from_top<PER, kCta>(own, (unsigned int)k, s_tot, s_out);
  if (threadIdx.x == 0) {
    ctl->Tbin = s_out[0];
    ctl->rem = s_out[1];
    ctl->by_bin = ctl->exact != 0 && s_out[0] + 1 < (unsigned int)kFineBins;
  }
}

}  // namespace nsml
