// Sampled lower bound for the top-k threshold (Alg. 2 Step 3: which
// k = ceil(ratio*n) gradients have the largest absolute value).
//
// The bucket is streamed exactly once, by the compaction pass, which needs a
// key `lo` such that a little more than k keys are >= lo.  k_sample draws one
// element from each of 8192 equal strata of the bucket and radix-selects the
// sample key whose rank leaves a six-sigma margin above the expected rank of
// the k-th largest; lo is that key rounded down to its top 24 bits.  The exact
// threshold is found afterwards on the short candidate list
// (nsml_finalize.cuh), which also repairs the rare case of a misleading
// sample, so the sample only decides how much work is done, never the result.
//
// The kernel is one cluster of eight blocks: 8192 threads fetch one scattered
// element each (one round of memory latency, spread over eight SMs), write the
// keys into block 0's shared memory through the cluster's distributed shared
// memory, meet at the cluster barrier, and block 0 selects.
#pragma once

#include <cooperative_groups.h>

#include "nsml_common.cuh"

namespace nsml {

constexpr int kSampleThreads = 1024;
constexpr int kSampleBlocks = 8;
constexpr int kSamples = kSampleThreads * kSampleBlocks;  // 8192 strata

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

// Clears the per-call control region and sets ctl->lo from a stratified
// sample of the bucket (of bucket + addend when an addend is given).  rank_from_top == 0 means "no sampling" (small bucket, or nearly
// everything is kept): lo = 0.
template <int DTYPE>
__global__ void __cluster_dims__(kSampleBlocks, 1, 1) __launch_bounds__(kSampleThreads)
k_sample(BucketSrc<DTYPE> src, const float* __restrict__ addend, unsigned long long n, unsigned int rank_from_top,
         Ctl* ctl, uint4* zero_base, unsigned int zero_vec16, int keep_status) {
  namespace cg = cooperative_groups;
  __shared__ unsigned int s_keys[kSamples];  // block 0: the sample keys, then (first 4096 words) the histogram
  unsigned int* s_hist = s_keys;
  __shared__ unsigned int s_tot[kSampleThreads / 32];
  __shared__ unsigned int s_out[2];
  cg::cluster_group cluster = cg::this_cluster();
  const unsigned int rank = cluster.block_rank();

  if (rank_from_top != 0) {
    const unsigned long long stratum = (unsigned long long)rank * kSampleThreads + threadIdx.x;
    const unsigned long long begin = stratum * n / kSamples;
    const unsigned long long end = (stratum + 1) * n / kSamples;  // > begin because n >= 2 * kSamples
    const unsigned long long pos = begin + mix32((uint32_t)stratum * 0x9E3779B1u + 0x85EBCA6Bu) % (uint32_t)(end - begin);
    // with an addend (the residual of the local accumulation) the bucket that is selected from is the sum
    uint32_t bits = src.load1(pos);
    if (addend != nullptr && !src.pruned(pos)) bits = __float_as_uint(__fadd_rn(__uint_as_float(src.raw1(pos)), addend[pos]));
    const uint32_t key = bits & 0x7FFFFFFFu;
    unsigned int* remote = cluster.map_shared_rank(s_keys, 0);
    remote[stratum] = key;
  }
  // keep_status: an error an earlier step of the same call left in the status word stays visible
  for (unsigned int i = rank * kSampleThreads + threadIdx.x; i < zero_vec16; i += kSamples)
    zero_base[i] = make_uint4((i == 0 && keep_status) ? (unsigned int)ctl->status : 0u, 0, 0, 0);
  cluster.sync();  // release/acquire at cluster scope: keys have landed in block 0, the control region is cleared
  if (rank != 0) return;

  unsigned int lo = 0;
  if (rank_from_top != 0) {
    uint32_t keys[kSampleBlocks];
#pragma unroll
    for (int s = 0; s < kSampleBlocks; ++s) keys[s] = s_keys[s * kSampleThreads + threadIdx.x];
    __syncthreads();  // every key is in registers: the buffer becomes the histogram
    unsigned int prefix = 0, rem = rank_from_top;
#pragma unroll
    for (int level = 0; level < 2; ++level) {  // 12 + 12 bits
      const int shift = digit_shift(level);
      __syncthreads();  // the previous level's bins have been read
      for (int b = threadIdx.x; b < kMaxBins; b += kSampleThreads) s_hist[b] = 0;
      __syncthreads();
#pragma unroll
      for (int s = 0; s < kSampleBlocks; ++s)
        if (level == 0 || (keys[s] >> 19) == prefix) atomicAdd(&s_hist[(keys[s] >> shift) & (kMaxBins - 1)], 1u);
      __syncthreads();
      unsigned int own[4];
#pragma unroll
      for (int b = 0; b < 4; ++b) own[b] = s_hist[threadIdx.x * 4 + b];
      find_digit_from_top<4, kSampleThreads>(own, rem, s_tot, s_out);
      prefix = (prefix << 12) | s_out[0];
      rem = s_out[1];
    }
    lo = prefix << 7;
  }
  if (threadIdx.x == 0) ctl->lo = lo;
}

}  // namespace nsml
