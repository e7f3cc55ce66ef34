// Helpers shared by the two cooperative kernels that turn a bucket into a
// payload (nsml_pick.cuh: from the candidates the bucket pass marked;
// nsml_dense.cuh: by a radix select over the bucket itself): block-wide sums
// and scans, the bounded grid barrier, histogram flush and digit resolve, and
// the quantisation of the survivors (Alg. 2 Step 1 "quantize" for fp16; int8
// per block of 1024 survivors).
//
// Every barrier wait is bounded: when it runs out the block records
// NSML_ERR_TIMEOUT and leaves; the others then time out as well.
#pragma once

#include "nsml_codec.cuh"
#include "nsml_common.cuh"
#include "nsml_select.cuh"

namespace nsml {

// Shapes of the dense select.  The small one (256 threads, 8192 cached values, ~53 KB of shared memory)
// is for buckets that fit it with one block per SM; the large one (two 512-thread blocks per SM hold
// 2 x 23040 values, 6.8M elements over 148 SMs: a 25 MB float32 bucket stays on chip) for the rest.
constexpr int kFinSmallThreads = 256, kFinSmallCache = 8192;
constexpr int kFinLargeThreads = 512;
constexpr int kFinDenseLargeCache = 23040;
constexpr size_t finalize_dyn_smem(int cache_entries) { return (size_t)cache_entries * 4; }  // values only

struct FinalizeParams {
  unsigned long long n, k;
  int bits;
  unsigned long long nseg;           // ceil(n / kSegElems)
  Ctl* ctl;
  unsigned int* hist;                // [4][kMaxBins]
  unsigned long long* block_counts;  // [4][kMaxFinalizeBlocks]
  float* raw_val;
  unsigned char* payload;
  PayloadLayout P;
  unsigned int dense_cache;          // values a block of the dense select keeps in shared memory (a multiple of 128)
  // list stage only
  const uint32_t* bitmap;
  uint2* und;                        // [kUndCap]
  unsigned int* qcount;
  unsigned int pick_blocks;          // blocks of the list kernels: ceil(n / kPickElems)
  unsigned int* per_block;           // [6][pick_blocks], see CompressLayout
  uint32_t* stash_val;               // [pick_blocks * kStashPerBlock]
  int only_on_fallback;              // dense select: leave at once unless the list stage asked for it
};

constexpr int kUndWarpCap = 192;  // undecided entries a warp of the dense select can list

template <int THREADS>
struct FinalizeShared {
  unsigned int hist[kMaxBins];
  unsigned short und[THREADS / 32][kUndWarpCap];
  unsigned long long red[(THREADS / 32)];
  unsigned long long run[2 * (THREADS / 32)];  // write phase: survivors per (warp, run)
  unsigned int scan[(THREADS / 32)];
  unsigned int tot[(THREADS / 32)];
  unsigned int out[2];
  float qmax[(THREADS / 32)];
  int ok;
};

// Sum over the block; every thread gets the result.
template <int THREADS>
__device__ __forceinline__ unsigned long long block_sum(unsigned long long v, FinalizeShared<THREADS>& sh) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  __syncthreads();  // sh.red may still be read from an earlier call
  if ((threadIdx.x & 31) == 0) sh.red[threadIdx.x >> 5] = v;
  __syncthreads();
  unsigned long long s = 0;
#pragma unroll
  for (int w = 0; w < (THREADS / 32); ++w) s += sh.red[w];
  return s;
}

// Exclusive prefix over the block in thread order; `total` = sum over the block.
template <int THREADS>
__device__ __forceinline__ unsigned int block_excl_scan(unsigned int v, unsigned int& total, FinalizeShared<THREADS>& sh) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  unsigned int incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned int up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
    if (lane >= o) incl += up;
  }
  __syncthreads();  // sh.scan may still be read from an earlier call
  if (lane == 31) sh.scan[warp] = incl;
  __syncthreads();
  unsigned int before = 0, all = 0;
#pragma unroll
  for (int w = 0; w < (THREADS / 32); ++w) {
    const unsigned int c = sh.scan[w];
    if (w < warp) before += c;
    all += c;
  }
  total = all;
  return before + incl - v;
}

// All blocks arrive, then all leave.  `target` = barrier ordinal * gridDim.x.
// CLUSTER: the grid is one thread-block cluster and the barrier is the hardware's (release / acquire at
// cluster scope, which orders the blocks' global-memory traffic as well); it cannot time out.
// SH: any shared-memory struct with an int member `ok`.  max_polls: polls after which the wait gives up.
template <bool CLUSTER = false, class SH>
__device__ __forceinline__ bool grid_barrier(Ctl* ctl, unsigned int target, SH& sh, int max_polls = kMaxPolls) {
  if (CLUSTER) {
    cooperative_groups::this_cluster().sync();
    return true;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    // Arrive with release, wait with acquire (both at device scope): what the block wrote before the
    // __syncthreads above is visible to every block that leaves the wait, without full fences.
    asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(&ctl->barrier), "r"(1u) : "memory");
    int ok = 1, polls = 0;
    for (;;) {
      unsigned int seen;
      asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(&ctl->barrier) : "memory");
      if (seen >= target) break;
      if (++polls > max_polls) { ok = 0; break; }
      if (polls > 256) __nanosleep(64);
    }
    if (!ok) set_status(&ctl->status, NSML_ERR_TIMEOUT);
    sh.ok = ok;
  }
  __syncthreads();
  return sh.ok != 0;
}

// Self-test of the bounded wait: every block arrives once at a barrier whose target is one arrival more
// than the grid can deliver, so each wait runs out after max_polls polls, the status word becomes
// NSML_ERR_TIMEOUT and the kernel returns by itself.
struct BarrierProbeShared { int ok; };
__global__ void __launch_bounds__(32) k_barrier_probe(Ctl* ctl, int max_polls) {
  __shared__ BarrierProbeShared sh;
  grid_barrier(ctl, gridDim.x + 1u, sh, max_polls);
}

// Adds the block's shared histogram into the global one (non-empty bins only).
template <int NB, int THREADS>
__device__ __forceinline__ void flush_hist(FinalizeShared<THREADS>& sh, unsigned int* ghist) {
  __syncthreads();
  for (int b = threadIdx.x; b < NB; b += THREADS) {
    const unsigned int c = sh.hist[b];
    if (c) atomicAdd(&ghist[b], c);
  }
}

// Every block reads the global histogram of a level and finds the digit that
// holds the rem-th largest key; digit and the rank left inside land in sh.out.
template <int NB, int THREADS>
__device__ __forceinline__ void resolve_digit(const unsigned int* ghist, unsigned int rem, FinalizeShared<THREADS>& sh) {
  constexpr int PER = (NB + THREADS - 1) / THREADS;
  unsigned int own[PER];
#pragma unroll
  for (int b = 0; b < PER; ++b) {
    const int bin = threadIdx.x * PER + b;
    own[b] = (bin < NB) ? __ldcg(ghist + bin) : 0u;
  }
  find_digit_from_top<PER, THREADS>(own, rem, sh.tot, sh.out);
}

// Clears the control block and the histograms of a workspace (what the sample
// kernel does on the list path) ahead of a dense-mode finalize.
__global__ void __launch_bounds__(kCta) k_clear(uint4* __restrict__ region, unsigned int count16, int keep_status) {
  for (unsigned int i = blockIdx.x * kCta + threadIdx.x; i < count16; i += gridDim.x * kCta)
    region[i] = make_uint4((i == 0 && keep_status) ? reinterpret_cast<const unsigned int*>(region)[0] : 0u, 0u, 0u, 0u);
}

__device__ __forceinline__ void write_header(const FinalizeParams& p) {
  nsml_payload_header h;
  h.magic = NSML_PAYLOAD_MAGIC;
  h.version = NSML_PAYLOAD_VERSION;
  h.n = p.n;
  h.k = p.k;
  h.bits = (uint32_t)p.bits;
  h.qblock = NSML_QBLOCK;
  h.nblocks = p.P.nblocks;
  h.idx_off = p.P.idx_off;
  h.val_off = p.P.val_off;
  h.scale_off = p.P.scale_off;
  *reinterpret_cast<nsml_payload_header*>(p.payload) = h;
}

// One round of the quantisation: thread group `threadIdx.x >> 8` (256 threads) converts the block of
// 1024 survivors qb from raw_val into the payload (int8 with a max-abs scale, fp16, or float32 as is);
// live = false: this group has no block this round.  Called by every thread of the thread block (it
// holds block barriers).
// SH: any shared-memory struct with a float array qmax of one entry per warp.
template <class SH>
__device__ __forceinline__ void quantize_block(const FinalizeParams& p, SH& sh, unsigned long long qb, bool live) {
  const int lane = threadIdx.x & 31;
  const int group = threadIdx.x >> 8, gtid = threadIdx.x & 255;
  const unsigned long long j0 = qb * NSML_QBLOCK + gtid * 4;
  float v[4] = {0.f, 0.f, 0.f, 0.f};
  int cnt = 0;
  if (live) {
    if (j0 + 4 <= p.k) {
      const float4 f = __ldcg(reinterpret_cast<const float4*>(p.raw_val + j0));
      v[0] = f.x; v[1] = f.y; v[2] = f.z; v[3] = f.w;
      cnt = 4;
    } else if (j0 < p.k) {
      cnt = (int)(p.k - j0);
      for (int e = 0; e < cnt; ++e) v[e] = __ldcg(p.raw_val + j0 + e);
    }
  }
  if (p.bits == NSML_BITS_FP32) {  // values travel as they are (Alg. 2 when Step 1 does not quantise)
    float* out = reinterpret_cast<float*>(p.payload + p.P.val_off);
    if (cnt == 4) {
      *reinterpret_cast<float4*>(out + j0) = make_float4(v[0], v[1], v[2], v[3]);
    } else {
      for (int e = 0; e < cnt; ++e) out[j0 + e] = v[e];
    }
    return;
  }
  if (p.bits == NSML_BITS_FP16) {
    uint16_t* out = reinterpret_cast<uint16_t*>(p.payload + p.P.val_off);
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
  // max-abs of the 1024 survivors: warp shuffles, then one value per warp through shared memory
  float m = fmaxf(fmaxf(fabsf(v[0]), fabsf(v[1])), fmaxf(fabsf(v[2]), fabsf(v[3])));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
  __syncthreads();  // qmax of the previous round has been read
  if (lane == 0) sh.qmax[threadIdx.x >> 5] = m;
  __syncthreads();
  m = sh.qmax[group * 8];
#pragma unroll
  for (int w = 1; w < 8; ++w) m = fmaxf(m, sh.qmax[group * 8 + w]);
  const float scale = __fdiv_rn(m, 127.0f);
  if (live) {
    if (gtid == 0) reinterpret_cast<float*>(p.payload + p.P.scale_off)[qb] = scale;
    signed char* out = reinterpret_cast<signed char*>(p.payload + p.P.val_off);
    if (cnt == 4) {
      uint32_t w = 0;
#pragma unroll
      for (int e = 0; e < 4; ++e) w |= ((uint32_t)encode_i8(v[e], scale) & 0xFFu) << (8 * e);
      *reinterpret_cast<uint32_t*>(out + j0) = w;
    } else {
      for (int e = 0; e < cnt; ++e) out[j0 + e] = (signed char)encode_i8(v[e], scale);
    }
  }
}

// Last phase of the dense select: quantises the k survivors left in raw_val into the payload, a group
// of 256 threads per block of 1024 survivors, and writes the payload header.
template <int THREADS>
__device__ __forceinline__ void quantize_phase(const FinalizeParams& p, FinalizeShared<THREADS>& sh) {
  const unsigned int G = gridDim.x, blk = blockIdx.x;
  if (blk == 0 && threadIdx.x == 0) write_header(p);
  const unsigned long long qblocks = (p.k + NSML_QBLOCK - 1) / NSML_QBLOCK;
  constexpr int kQGroups = THREADS / 256;
  for (unsigned long long q0 = (unsigned long long)blk * kQGroups; q0 < qblocks; q0 += (unsigned long long)G * kQGroups) {
    const unsigned long long qb = q0 + (threadIdx.x >> 8);
    quantize_block(p, sh, qb, qb < qblocks);
  }
}

}  // namespace nsml
