// Bucket -> segmented candidate list: the one full pass over the bucket
// (Alg. 2 Steps 2-3: pruned gradients read as zero; everything whose magnitude
// is below the sampled lower bound is dropped here, in one streaming read).
//
// Warp w owns a contiguous range of 128-element rounds and appends what it
// keeps (every key >= lo, lo >= 1) to its own segment of the list.  A segment
// starts at the list position of the range's first element, so it can never
// overflow and needs no allocation.  There is no block or grid
// synchronisation: a warp's only state is its running count.  Segments taken
// in warp order are in index order.
#pragma once

#include "nsml_common.cuh"

namespace nsml {

constexpr int kRound = 128;  // elements a warp handles per step (32 lanes x 4)
constexpr int kUnroll = 4;   // rounds in flight per warp

__host__ __device__ inline unsigned long long warp_first_round(unsigned long long warp, unsigned long long warps,
                                                               unsigned long long rounds) {
  return warp * rounds / warps;
}

// Appends the kept elements of one round.  `f` holds this lane's four keep
// flags (bit e = element lane*4+e of the round).  Returns the round's total.
__device__ __forceinline__ unsigned int append_round(unsigned int f, const uint32_t (&bits)[4], uint32_t first_index,
                                                     unsigned long long out_base, uint32_t* __restrict__ seg_idx,
                                                     uint32_t* __restrict__ seg_val) {
  const int lane = threadIdx.x & 31;
  const unsigned int lt = (1u << lane) - 1u;
  const unsigned int any = __ballot_sync(0xFFFFFFFFu, f != 0);
  const unsigned int multi = __ballot_sync(0xFFFFFFFFu, (f & (f - 1)) != 0);
  unsigned int before, total;
  if (multi == 0) {  // usual case: no lane keeps more than one element
    before = __popc(any & lt);
    total = __popc(any);
  } else {
    const unsigned int mine = __popc(f);
    unsigned int incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned int up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
      if (lane >= o) incl += up;
    }
    before = incl - mine;
    total = __shfl_sync(0xFFFFFFFFu, incl, 31);
  }
  if (f != 0) {
    unsigned long long pos = out_base + before;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      if (f & (1u << e)) {
        seg_idx[pos] = first_index + lane * 4 + e;
        seg_val[pos] = bits[e];
        ++pos;
      }
    }
  }
  return total;
}

template <int DTYPE>
__global__ void __launch_bounds__(kCta)
k_compact_bucket(BucketSrc<DTYPE> src, unsigned long long n, Ctl* ctl, uint32_t* __restrict__ seg_idx,
                 uint32_t* __restrict__ seg_val, unsigned int* __restrict__ seg_count) {
  const int lane = threadIdx.x & 31;
  const unsigned long long warp = (unsigned long long)blockIdx.x * (kCta / 32) + (threadIdx.x >> 5);
  const unsigned long long warps = (unsigned long long)gridDim.x * (kCta / 32);
  const unsigned long long rounds = (n + kRound - 1) / kRound;
  const unsigned long long first = warp_first_round(warp, warps, rounds);
  const unsigned long long last = warp_first_round(warp + 1, warps, rounds);
  // Zeros are never candidates here; if they are needed (fewer than k non-zero
  // keys) the list comes out short and the finalize kernel's slow path adds them.
  // |v| >= t on floats equals key >= lo for finite v; written as !(|v| < t) so
  // that NaN is kept too (the finalize kernel reports non-finite candidates).
  const float t = __uint_as_float(max(ctl->lo, 1u));
  const unsigned long long seg_base = first * kRound;
  const unsigned long long full_rounds = n / kRound;  // rounds that need no bounds checks
  unsigned int kept = 0;

  unsigned long long rd = first;
  const unsigned long long last_full = min(last, full_rounds);
  for (; rd + kUnroll <= last_full; rd += kUnroll) {
    uint32_t bits[kUnroll][4];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) src.load_full4((rd + u) * kRound + lane * 4, bits[u]);
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      unsigned int f = 0;
#pragma unroll
      for (int e = 0; e < 4; ++e) f |= (unsigned)(!(fabsf(__uint_as_float(bits[u][e])) < t)) << e;
      if (!__any_sync(0xFFFFFFFFu, f != 0)) continue;
      kept += append_round(f, bits[u], (uint32_t)((rd + u) * kRound), seg_base + kept, seg_idx, seg_val);
    }
  }
  for (; rd < last; ++rd) {  // leftover rounds, the last of which may be partial
    uint32_t bits[4];
    src.load_vals4(rd * kRound + lane * 4, n, bits);  // missing elements read as 0 and are never kept
    unsigned int f = 0;
#pragma unroll
    for (int e = 0; e < 4; ++e) f |= (unsigned)(!(fabsf(__uint_as_float(bits[e])) < t)) << e;
    if (!__any_sync(0xFFFFFFFFu, f != 0)) continue;
    kept += append_round(f, bits, (uint32_t)(rd * kRound), seg_base + kept, seg_idx, seg_val);
  }
  if (lane == 0) seg_count[warp] = kept;
}

}  // namespace nsml
