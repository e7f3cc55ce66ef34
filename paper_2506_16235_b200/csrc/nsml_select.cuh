// Sampled bracket for the top-k threshold (Alg. 2 Step 3: which
// k = ceil(ratio*n) gradients have the largest absolute value).
//
// The bucket is streamed exactly once, by the bucket pass, which needs a key
// `lo` such that a little more than k keys are >= lo.  k_sample draws one
// element from each of 8192 equal strata of the bucket and radix-selects two
// sample keys: the one whose rank leaves a six-sigma margin above the expected
// rank of the k-th largest (lo, rounded down to its top 24 bits) and the one
// six sigma below it (hi).  The exact threshold lies between the two unless
// the sample misleads; the bucket pass counts the candidates (keys >= lo) in
// kFineBins key bins whose width is chosen here so that [lo, hi] spans three
// quarters of them.  The exact threshold is found afterwards among the
// candidates (nsml_pick.cuh), which also repairs the rare case of a misleading
// sample, so the sample only decides how much work is done, never the result.
//
// The kernel is one cluster of eight blocks: every thread fetches one
// scattered element (one round of memory latency, spread over eight SMs) and
// writes its key into block 0's shared memory through the cluster's
// distributed shared memory; after one cluster barrier block 0 selects.
#pragma once

#include <cooperative_groups.h>

#include "nsml_common.cuh"

namespace nsml {

constexpr int kSampleThreads = 1024;
constexpr int kSampleBlocks = 8;
constexpr int kSamplePer = 1;  // scattered elements a thread fetches
constexpr int kSamples = kSampleThreads * kSampleBlocks * kSamplePer;  // 8192 strata

__device__ __forceinline__ uint32_t mix32(uint32_t x) {
  x ^= x >> 16; x *= 0x7FEB352Du;
  x ^= x >> 15; x *= 0x846CA68Bu;
  x ^= x >> 16;
  return x;
}

// Block-wide search from the top over bins held PER per thread (own[] holds
// this thread's consecutive bins, lowest first): leaves in s_out the digit d
// with #{digit > d} < rem <= #{digit >= d} and the rank left inside bin d.
// Called by every thread of the block; s_tot needs one word per warp.
template <int PER, int THREADS>
__device__ __forceinline__ void find_digit_from_top(const unsigned int (&own)[PER], unsigned int rem,
                                                    unsigned int* s_tot, unsigned int* s_out) {
  const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
  unsigned int mine = 0;
#pragma unroll
  for (int b = 0; b < PER; ++b) mine += own[b];
  unsigned int incl = mine;  // this thread and all higher lanes of the warp
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned int v = __shfl_down_sync(0xFFFFFFFFu, incl, o);
    if (lane + o < 32) incl += v;
  }
  __syncthreads();  // s_tot and s_out may still be read from an earlier call
  if (lane == 0) s_tot[warp] = incl;
  __syncthreads();
  unsigned int above = incl - mine;
  for (int w = warp + 1; w < THREADS / 32; ++w) above += s_tot[w];
  if (above < rem && rem <= above + mine) {  // exactly one thread
#pragma unroll
    for (int b = PER - 1; b >= 0; --b) {
      if (rem <= above + own[b]) {
        s_out[0] = (unsigned)(t * PER + b);
        s_out[1] = rem - above;
        break;
      }
      above += own[b];
    }
  }
  __syncthreads();
}

// Clears the per-call control region and sets ctl->lo, ctl->shift and ctl->exact from a stratified
// sample of the bucket (of bucket + addend when an addend is given).  rank_lo / rank_hi: ranks from the
// top (1-based) of the two sample keys that bracket the threshold.  keys16: the keys that
// are selected from are bfloat16 magnitudes (their low 16 bits are zero), so a bin of width 2^16 holds
// one key value.  keep_status: an error an earlier step of the same call left in the status word stays.
constexpr size_t kSampleSmem = (size_t)kSamples * sizeof(uint32_t);  // dynamic shared memory of k_sample: block 0 holds every key

template <int DTYPE>
__global__ void __cluster_dims__(kSampleBlocks, 1, 1) __launch_bounds__(kSampleThreads)
k_sample(BucketSrc<DTYPE> src, const float* __restrict__ addend, unsigned long long n, unsigned int rank_lo,
         unsigned int rank_hi, int keys16, Ctl* ctl, uint4* zero_base, unsigned int zero_vec16, int keep_status) {
  namespace cg = cooperative_groups;
  extern __shared__ __align__(16) uint32_t s_keys[];  // block 0: the sample keys of all eight blocks
  __shared__ __align__(16) unsigned int s_hist_lo[kMaxBins];  // keys by first digit; then: by second digit under lo's first digit
  __shared__ __align__(16) unsigned int s_hist_hi[kMaxBins];  // keys by second digit under hi's first digit
  __shared__ unsigned int s_tot[kSampleThreads / 32];
  __shared__ unsigned int s_out[2];
  cg::cluster_group cluster = cg::this_cluster();
  const unsigned int rank = cluster.block_rank();
  const int t = threadIdx.x;

  uint32_t mine[kSamplePer];
  const unsigned long long width = n / kSamples;  // >= 2; the last stratum also takes the remainder, which is never sampled
#pragma unroll
  for (int s = 0; s < kSamplePer; ++s) {
    const unsigned int stratum = ((unsigned int)s * kSampleBlocks + rank) * kSampleThreads + t;
    // a hashed offset inside the stratum: the high word of hash * width
    const unsigned long long pos = (unsigned long long)stratum * width +
                                   (((unsigned long long)mix32(stratum * 0x9E3779B1u + 0x85EBCA6Bu) * width) >> 32);
    // with an addend (the residual of the local accumulation) the bucket that is selected from is the sum
    uint32_t bits = src.load1(pos);
    if (addend != nullptr && !src.pruned(pos)) bits = __float_as_uint(__fadd_rn(__uint_as_float(src.raw1(pos)), addend[pos]));
    mine[s] = bits & 0x7FFFFFFFu;
  }
  // while the loads are in flight everybody clears the control region
  for (unsigned int i = rank * kSampleThreads + t; i < zero_vec16; i += kSampleThreads * kSampleBlocks)
    zero_base[i] = make_uint4((i == 0 && keep_status) ? (unsigned int)ctl->status : 0u, 0, 0, 0);
  {
    uint32_t* all_keys = cluster.map_shared_rank(s_keys, 0);
#pragma unroll
    for (int s = 0; s < kSamplePer; ++s) all_keys[((unsigned int)s * kSampleBlocks + rank) * kSampleThreads + t] = mine[s];
  }
  cluster.sync();  // release/acquire at cluster scope: the keys have landed in block 0, the control region is cleared
  if (rank != 0) return;

  constexpr int PER_THREAD = kSamples / kSampleThreads;  // 8
  unsigned int prefix_lo = 0, prefix_hi = 0, rem_lo = rank_lo, rem_hi = rank_hi;
#pragma unroll
  for (int level = 0; level < 2; ++level) {  // 12 + 12 bits
    const int shift = digit_shift(level);
    for (int b = t; b < kMaxBins; b += kSampleThreads) {
      s_hist_lo[b] = 0;
      s_hist_hi[b] = 0;
    }
    __syncthreads();
#pragma unroll 8
    for (int s = 0; s < PER_THREAD; ++s) {
      const uint32_t key = s_keys[s * kSampleThreads + t];
      const unsigned int bin = (key >> shift) & (kMaxBins - 1);
      if (level == 0 || (key >> 19) == prefix_lo) atomicAdd(&s_hist_lo[bin], 1u);
      if (level == 1 && (key >> 19) == prefix_hi) atomicAdd(&s_hist_hi[bin], 1u);
    }
    __syncthreads();
    unsigned int own[4];
    {
      const uint4 v = reinterpret_cast<const uint4*>(s_hist_lo)[t];
      own[0] = v.x; own[1] = v.y; own[2] = v.z; own[3] = v.w;
    }
    find_digit_from_top<4, kSampleThreads>(own, rem_lo, s_tot, s_out);
    prefix_lo = (prefix_lo << 12) | s_out[0];
    rem_lo = s_out[1];
    if (level == 1) {
      const uint4 h = reinterpret_cast<const uint4*>(s_hist_hi)[t];
      own[0] = h.x; own[1] = h.y; own[2] = h.z; own[3] = h.w;
    }
    find_digit_from_top<4, kSampleThreads>(own, rem_hi, s_tot, s_out);
    prefix_hi = (prefix_hi << 12) | s_out[0];
    rem_hi = s_out[1];
  }
  if (t != 0) return;
  const unsigned int lo = prefix_lo << 7;
  // first key above hi's 24-bit class
  const unsigned int hi = (prefix_hi + 1u) << 7;
  const unsigned int span = hi > lo ? hi - lo : 0u;
  unsigned int shift = 0;
  while ((span >> shift) >= (unsigned int)(kFineBins * 3 / 4)) ++shift;
  unsigned int exact = shift == 0;
  if (keys16) {  // bins narrower than one bfloat16 step would stay empty
    exact = shift <= 16;
    if (shift < 16) shift = 16;
  }
  ctl->lo = lo;
  ctl->shift = shift;
  ctl->exact = exact;
}

}  // namespace nsml
