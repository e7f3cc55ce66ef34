// Candidate list -> payload, in one cooperative kernel.
//
// The bucket pass leaves a segmented list of candidates (every key >= lo).
// This kernel finds the exact threshold key T and the tie budget r by radix
// select on the candidates' magnitude keys (12 + 12 + 7 bits; Alg. 2 Step 3
// read as: keep the k largest |g|, ties by lower index), writes the k
// survivors in index order and quantises them (Alg. 2 Step 1 "quantize" for
// fp16; int8 per block of 1024 survivors).
//
// All blocks are co-resident (cooperative launch).  k_gather (below) first
// makes the segmented list contiguous and counts the candidates' first key
// digit.  The bucket pass also leaves a candidate count per group of 64
// segments; every block of k_finalize scans those, which gives it the total,
// and takes an equal share of the contiguous list (so "index order" is block
// order, and the blocks' work is balanced however the candidates crowd).
// Phases, separated by grid barriers:
//   0  copy the share's values into shared memory as far as they fit
//   1  every block resolves digit 0 (from the gather's histogram);
//      histogram of digit 1                                                | barrier
//   2  resolve digit 1; histogram of digit 2                               | barrier
//   3  resolve digit 2 -> T, r; count own keys > T and == T                | barrier
//   4  prefix over blocks; write survivors in order: index, and the value
//      as float32 / fp16 directly or, for int8, parked in raw_val
//   5  block 0 writes the header; int8 only, behind one more barrier: quantise
//      blocks of 1024 survivors
// If the list holds fewer than k candidates (fewer than k non-zero keys, or a
// misleading sample) phase 0 is replaced by a slow path in which block b owns
// an index range and rebuilds its array from the bucket: every non-zero key
// plus the first k - nnz zeros in index order (one more barrier).
//
// Calls in which the list would be about as large as the bucket take k_finalize_dense
// (nsml_dense.cuh) instead, which shares this file's helpers and the quantise phase.
//
// Every barrier wait is bounded: when it runs out the block records
// NSML_ERR_TIMEOUT and leaves; the others then time out as well.
#pragma once

#include "nsml_codec.cuh"
#include "nsml_common.cuh"
#include "nsml_compact.cuh"
#include "nsml_select.cuh"

namespace nsml {

// Two shapes of the kernel.  The small one (256 threads, 8192 cached candidate
// values, ~53 KB of shared memory, 16K registers) lets several list stages, and the
// next bucket's streaming pass, share an SM when buckets are compressed on
// several streams; the large one is for long candidate lists.
constexpr int kFinSmallThreads = 256, kFinSmallCache = 8192;
constexpr int kFinLargeThreads = 512, kFinLargeCache = 20480;
// The shortest lists (a few candidates per thread) run as ONE thread-block cluster of kFinClusterBlocks
// blocks of 1024 threads: the barriers between the phases are the cluster's hardware barriers (a fraction
// of a microsecond instead of a round trip through global memory), and the rest of the GPU stays free for
// other streams' kernels.  Measured on a 6.5M-element bucket at ratio 0.001 (about 20k candidates): 42 us
// against 58 us for five 256-thread blocks; from about 50k candidates on the per-block copy work
// outweighs the cheaper barriers (110k candidates: 64 against 48 us).
constexpr int kFinClusterBlocks = 8, kFinClusterThreads = 1024, kFinClusterCache = 8192;
constexpr double kFinClusterMaxCandidates = 32768.0;  // expected candidates up to which the cluster shape is used
// The dense kernel needs no gather scratch, which leaves room for a larger cache in the large shape: two
// blocks per SM then hold 2 x 23040 values, 6.8M elements over 148 SMs (a 25 MB float32 bucket stays on chip).
constexpr int kFinDenseLargeCache = 23040;
constexpr size_t finalize_dyn_smem(int cache_entries) { return (size_t)cache_entries * 4; }  // values only

struct FinalizeParams {
  unsigned long long n, k;
  int bits;
  unsigned long long nseg;           // ceil(n / kSegElems)
  Ctl* ctl;
  unsigned int* hist;                // [4][kMaxBins]
  unsigned long long* block_counts;  // [4][kMaxFinalizeBlocks]
  const unsigned short* seg_count;
  const unsigned int* group_count;   // [ceil(nseg / kGroupSegs)]
  const unsigned short* seg_off;     // a candidate's offset inside its segment
  const uint32_t* seg_val;
  uint32_t* list_idx;
  uint32_t* list_val;
  float* raw_val;
  unsigned char* payload;
  PayloadLayout P;
};

template <int THREADS, bool DENSE>
struct GatherScratch {};  // the list kernel needs none: k_gather has made its list contiguous
constexpr int kUndCap = 192;  // undecided entries a warp of the dense kernel can list
template <int THREADS>
struct GatherScratch<THREADS, true> {  // the dense kernel gathers nothing; it lists undecided entries per warp
  unsigned short und[THREADS / 32][kUndCap];
};

template <int THREADS, bool DENSE>
struct FinalizeShared {
  unsigned int hist[kMaxBins];
  GatherScratch<THREADS, DENSE> g;
  unsigned long long red[(THREADS / 32)];
  unsigned long long run[2 * (THREADS / 32)];  // write phase: survivors per (warp, run)
  unsigned int scan[(THREADS / 32)];
  unsigned int tot[(THREADS / 32)];
  unsigned int out[2];
  float qmax[(THREADS / 32)];
  int ok;
};

// Sum over the block; every thread gets the result.
template <int THREADS, bool D>
__device__ __forceinline__ unsigned long long block_sum(unsigned long long v, FinalizeShared<THREADS, D>& sh) {
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
template <int THREADS, bool D>
__device__ __forceinline__ unsigned int block_excl_scan(unsigned int v, unsigned int& total, FinalizeShared<THREADS, D>& sh) {
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
template <int NB, int THREADS, bool D>
__device__ __forceinline__ void flush_hist(FinalizeShared<THREADS, D>& sh, unsigned int* ghist) {
  __syncthreads();
  for (int b = threadIdx.x; b < NB; b += THREADS) {
    const unsigned int c = sh.hist[b];
    if (c) atomicAdd(&ghist[b], c);
  }
}

// Every block reads the global histogram of a level and finds the digit that
// holds the rem-th largest key; digit and the rank left inside land in sh.out.
template <int NB, int THREADS, bool D>
__device__ __forceinline__ void resolve_digit(const unsigned int* ghist, unsigned int rem, FinalizeShared<THREADS, D>& sh) {
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

// A survivor's value on its way out: float32 and fp16 values go straight to their payload position (Alg. 2
// Step 1 "quantize" for fp16); int8 values are parked in raw_val until their block of 1024 is complete.
__device__ __forceinline__ void put_value(const FinalizeParams& p, unsigned long long pos, uint32_t bits) {
  if (p.bits == NSML_BITS_FP32) reinterpret_cast<uint32_t*>(p.payload + p.P.val_off)[pos] = bits;
  else if (p.bits == NSML_BITS_FP16) reinterpret_cast<uint16_t*>(p.payload + p.P.val_off)[pos] = encode_f16(__uint_as_float(bits));
  else p.raw_val[pos] = __uint_as_float(bits);
}

// int8: thread group `threadIdx.x >> 8` (256 threads) converts the block of 1024 survivors qb from raw_val
// into codes and a max-abs scale; live = false: this group has no block this round.  Called by every thread
// of the thread block (it holds block barriers).
template <int THREADS, bool D>
__device__ __forceinline__ void quantize_block(const FinalizeParams& p, FinalizeShared<THREADS, D>& sh, unsigned long long qb,
                                               bool live) {
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

// int8 only, after a grid barrier behind the write phase: every block of 1024 survivors parked in raw_val
// becomes codes and a scale, a group of 256 threads per block.  (Measured against letting whichever thread
// block delivers a payload block's last survivor quantise it, with no barrier: the atomic, the fences and the
// read-back cost that variant as much as the barrier costs this one, 34.9 against 33.2 us for the list stage
// of a 25M-element bucket.)
template <int THREADS, bool D>
__device__ __forceinline__ void quantize_all(const FinalizeParams& p, FinalizeShared<THREADS, D>& sh) {
  const unsigned long long qblocks = (p.k + NSML_QBLOCK - 1) / NSML_QBLOCK;
  constexpr int kQGroups = THREADS / 256;
  for (unsigned long long q0 = (unsigned long long)blockIdx.x * kQGroups; q0 < qblocks; q0 += (unsigned long long)gridDim.x * kQGroups) {
    const unsigned long long qb = q0 + (threadIdx.x >> 8);
    quantize_block(p, sh, qb, qb < qblocks);
  }
}

// Segmented candidate list -> contiguous list (list_idx / list_val, in index order) plus the global
// histogram of the candidates' first key digit.  A plain (non-cooperative) kernel that spreads the copy
// over all SMs: every candidate sits in another memory sector, and what bounds the copy is the rate of
// scattered loads per SM.  A block takes kGatherSegs consecutive segments (one group); the list
// position of its first candidate is the sum of the group counts before it; inside the block the
// candidates are taken entry-parallel (thread t copies entries t*4..t*4+3, t*4 + 4*256.., located by a
// search over the segments' offsets), so crowded segments are shared by all threads.
constexpr int kGatherSegs = kGroupSegs;  // one group per block: its list position is a plain sum of group counts
constexpr int kGatherRun = 4;      // consecutive candidates a thread copies per step
constexpr int kGatherBins = 256;   // first-digit bins a block of the gather counts in shared memory
constexpr int kGatherThreads = 128;  // threads per block (at least kGatherSegs)

// `split` blocks share a group (block b takes group b / split and every split-th step of its entries), so
// that long lists and crowded groups are spread over more blocks.
__global__ void __launch_bounds__(kGatherThreads)
k_gather(FinalizeParams p, unsigned int split) {
  // Every candidate's key is >= the sampled bound lo, and almost all lie within a few octaves above it:
  // the block counts first digits in a window of kGatherBins bins that starts at lo's bin (16 bins per
  // octave); the rare key beyond the window goes to the global histogram directly.
  __shared__ unsigned int s_hist[kGatherBins];
  __shared__ unsigned int s_off[kGatherSegs + 1];  // exclusive offsets of the block's segments, total at the end
  __shared__ unsigned long long s_red[kGatherThreads / 32];
  __shared__ unsigned int s_scan[kGatherThreads / 32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int b = threadIdx.x; b < kGatherBins; b += kGatherThreads) s_hist[b] = 0;
  const unsigned int first_bin = p.ctl->lo >> digit_shift(0);
  // list position of the block's first candidate
  const unsigned int group = blockIdx.x / split, part = blockIdx.x % split;
  const unsigned long long first_group = (unsigned long long)group * (kGatherSegs / kGroupSegs);
  unsigned long long before = 0;
  for (unsigned long long g = threadIdx.x; g < first_group; g += kGatherThreads) before += p.group_count[g];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) before += __shfl_xor_sync(0xFFFFFFFFu, before, o);
  if (lane == 0) s_red[warp] = before;
  // offsets of the block's segments
  const unsigned long long seg0 = (unsigned long long)group * kGatherSegs;
  const unsigned long long seg = seg0 + threadIdx.x;
  const unsigned int c = (threadIdx.x < kGatherSegs && seg < p.nseg) ? p.seg_count[seg] : 0u;
  unsigned int incl = c;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned int up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
    if (lane >= o) incl += up;
  }
  if (lane == 31) s_scan[warp] = incl;
  __syncthreads();
  unsigned long long base = 0;
  unsigned int warps_before = 0, total = 0;
#pragma unroll
  for (int w = 0; w < kGatherThreads / 32; ++w) {
    base += s_red[w];
    if (w < warp) warps_before += s_scan[w];
    total += s_scan[w];
  }
  if (threadIdx.x < kGatherSegs) s_off[threadIdx.x] = warps_before + incl - c;
  if (threadIdx.x == 0) s_off[kGatherSegs] = total;
  __syncthreads();
  bool nonfinite = false;
  for (unsigned int j0 = (part * kGatherThreads + threadIdx.x) * kGatherRun; j0 < total; j0 += split * kGatherThreads * kGatherRun) {
    const int cnt = (int)min((unsigned int)kGatherRun, total - j0);
    uint32_t from[kGatherRun];
    {
      // segment of entry j0: the last one whose offset is <= j0 (empty segments share an offset with their
      // successor, so the search lands on the segment that holds the entry)
      int lo = 0, hi = kGatherSegs - 1;
      while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (s_off[mid] <= j0) lo = mid; else hi = mid - 1;
      }
      unsigned int q = lo, within = j0 - s_off[lo];
#pragma unroll
      for (int e = 0; e < kGatherRun; ++e) {
        from[e] = 0;
        if (e < cnt) {
          while (within >= s_off[q + 1] - s_off[q]) { within = 0; ++q; }  // entry e exists, so this ends inside the block
          from[e] = (uint32_t)((seg0 + q) * kSegElems + within);
          ++within;
        }
      }
    }
    uint32_t vals[kGatherRun], idxs[kGatherRun];
#pragma unroll
    for (int e = 0; e < kGatherRun; ++e) {
      if (e < cnt) {
        vals[e] = __ldg(p.seg_val + from[e]);
        idxs[e] = (from[e] & ~(uint32_t)(kSegElems - 1)) + __ldg(p.seg_off + from[e]);
      }
    }
#pragma unroll
    for (int e = 0; e < kGatherRun; ++e) {
      if (e < cnt) {
        const uint32_t key = vals[e] & 0x7FFFFFFFu;
        p.list_idx[base + j0 + e] = idxs[e];
        p.list_val[base + j0 + e] = vals[e];
        nonfinite |= key >= kInfKey;
        const unsigned int bin = key >> digit_shift(0), rel = bin - first_bin;  // wraps only for a key below lo
        if (rel < (unsigned int)kGatherBins) atomicAdd(&s_hist[rel], 1u);
        else atomicAdd(&p.hist[bin], 1u);
      }
    }
  }
  if (nonfinite) set_status(&p.ctl->status, NSML_ERR_NONFINITE);
  __syncthreads();
  for (int b = threadIdx.x; b < kGatherBins; b += kGatherThreads) {
    const unsigned int n_b = s_hist[b];
    if (n_b) atomicAdd(&p.hist[first_bin + b], n_b);  // first_bin + b <= 4095: a count here came from a real key
  }
}

// Registers: at most 64 per thread; the small shape is held to 48 (five blocks per SM by registers, no spills).
// The kernel waits for memory most of its time, and what it costs other streams' kernels is the registers it
// holds meanwhile: with 48 instead of 64 the eight-stream step of the default workload went from 0.722 to
// 0.702 ms at the same time for a lone call (40: 0.704 ms with a few spills, 32: 0.719 ms and 6 us more alone).
// The large shape (two 512-thread blocks per SM) is held to 40: at 64 its grid took every register of every SM
// for the length of the kernel (ratio 0.1 on 25M-element buckets: 884 -> 921 GB/s, the kernel alone 47 -> 49 us).
template <int DTYPE, int THREADS, int CACHE, bool CLUSTER = false>
__global__ void __launch_bounds__(THREADS, THREADS == 256 ? 5 : (THREADS == 512 ? 3 : 1))
k_finalize(BucketSrc<DTYPE> src, FinalizeParams p) {
  __shared__ FinalizeShared<THREADS, false> sh;
  extern __shared__ __align__(16) uint32_t s_cache[];  // the first CACHE candidate values of this block
  uint32_t* cache_val = s_cache;
  const int lane = threadIdx.x & 31;
  const unsigned int G = gridDim.x, blk = blockIdx.x;
  // Index-range ownership (used by the slow path only) and the block's array.
  const unsigned long long seg_first = (unsigned long long)blk * p.nseg / G;
  const unsigned long long seg_last = (unsigned long long)(blk + 1) * p.nseg / G;
  uint32_t* my_idx = p.list_idx;  // set below
  uint32_t* my_val = p.list_val;
  unsigned int barriers = 0;
  unsigned int E = 0;  // candidates this block owns

  auto entry_val = [&](unsigned int j) -> uint32_t { return j < (unsigned)CACHE ? cache_val[j] : __ldcg(my_val + j); };
  auto put_entry = [&](unsigned int j, uint32_t idx, uint32_t val) {
    my_idx[j] = idx;  // indices are needed once, at the end: they stay in global memory
    if (j < (unsigned)CACHE) cache_val[j] = val; else my_val[j] = val;
  };

  // Calls f(key) for each of the block's candidates, four loads in flight per thread (the values beyond the
  // shared-memory cache come from global memory, where one load at a time would cost a round trip each).
  auto for_each_key = [&](auto f) {
    for (unsigned int j0 = threadIdx.x; j0 < E; j0 += THREADS * 4) {
      uint32_t v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const unsigned int j = j0 + u * THREADS;
        v[u] = (j < E) ? entry_val(j) : 0u;
      }
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (j0 + u * THREADS < E) f(v[u] & 0x7FFFFFFFu);
    }
  };

  // ---------------- phase 0: take an equal share of the candidates, histogram of digit 0 ----------------
  const unsigned int* ghist0 = p.hist;
  for (int b = threadIdx.x; b < kMaxBins; b += THREADS) sh.hist[b] = 0;
  bool nonfinite = false;
  {
    // Every block reads the per-group candidate counts the bucket pass left and
    // scans them, which gives the list position of every group and the total.
    const unsigned long long ngroups = (p.nseg + kGroupSegs - 1) / kGroupSegs;
    const unsigned long long per_thread = (ngroups + THREADS - 1) / THREADS;
    const unsigned long long g_begin = min(ngroups, threadIdx.x * per_thread);
    const unsigned long long g_end = min(ngroups, g_begin + per_thread);
    unsigned long long thread_sum = 0;
    for (unsigned long long gi = g_begin; gi < g_end; ++gi) thread_sum += p.group_count[gi];
    unsigned long long list_total;
    unsigned long long thread_pos;  // list position where this thread's first group starts
    {
      // 64-bit exclusive scan over the block
      const int warp = threadIdx.x >> 5;
      unsigned long long incl = thread_sum;
  #pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += up;
      }
      if (lane == 31) sh.red[warp] = incl;
      __syncthreads();
      unsigned long long before = 0, all = 0;
  #pragma unroll
      for (int w = 0; w < (THREADS / 32); ++w) {
        const unsigned long long c = sh.red[w];
        if (w < warp) before += c;
        all += c;
      }
      list_total = all;
      thread_pos = before + incl - thread_sum;
    }
    const unsigned long long share_lo = (unsigned long long)blk * list_total / G;
    const unsigned long long share_hi = (unsigned long long)(blk + 1) * list_total / G;
    if (list_total >= p.k) {
      my_idx = p.list_idx + share_lo;
      my_val = p.list_val + share_lo;
      E = (unsigned int)(share_hi - share_lo);
      // k_gather has made the list contiguous and built the histogram of digit 0: the block's share is a
      // plain range of it; its first CACHE values are copied into shared memory for the phases below.
      for (unsigned int j = threadIdx.x; j < min(E, (unsigned int)CACHE); j += THREADS) cache_val[j] = __ldcg(my_val + j);
    }

    if (list_total < p.k) {
      // ---- slow path: this block's array becomes (all non-zero keys) + (zeros within budget) ----
      const unsigned long long r_lo = seg_first * (unsigned long long)kSegElems;
      const unsigned long long r_hi = min(seg_last * (unsigned long long)kSegElems, p.n);
      my_idx = p.list_idx + r_lo;  // a block's range has room for all of its elements
      my_val = p.list_val + r_lo;
      unsigned long long nnz = 0, zeros = 0;
      for (unsigned long long i0 = r_lo + threadIdx.x * 4ull; i0 < r_hi; i0 += THREADS * 4ull) {
        uint32_t bits[4];
        const int cnt = src.load_vals4(i0, p.n, bits);
  #pragma unroll
        for (int e = 0; e < 4; ++e) {
          if (e < cnt) {
            if ((bits[e] & 0x7FFFFFFFu) != 0) ++nnz; else ++zeros;
          }
        }
      }
      const unsigned long long block_nnz = block_sum(nnz, sh);
      const unsigned long long block_zeros = block_sum(zeros, sh);
      unsigned long long* nz_counts = p.block_counts + 2 * kMaxFinalizeBlocks;
      if (threadIdx.x == 0) nz_counts[blk] = (block_nnz << 32) | block_zeros;
      if (!grid_barrier<CLUSTER>(p.ctl, ++barriers * G, sh)) return;

      unsigned long long all_nnz = 0, zeros_before = 0;
      for (unsigned int b = threadIdx.x; b < G; b += THREADS) {
        const unsigned long long w = __ldcg(nz_counts + b);
        all_nnz += w >> 32;
        if (b < blk) zeros_before += w & 0xFFFFFFFFull;
      }
      all_nnz = block_sum(all_nnz, sh);
      zeros_before = block_sum(zeros_before, sh);
      const unsigned long long zero_budget = (p.k > all_nnz) ? p.k - all_nnz : 0;
      // zeros of this block to keep, lowest index first
      const unsigned long long allowed = (zero_budget > zeros_before) ? min(block_zeros, zero_budget - zeros_before) : 0ull;

      __syncthreads();
      for (int b = threadIdx.x; b < kMaxBins; b += THREADS) sh.hist[b] = 0;
      E = 0;
      unsigned long long zeros_seen = 0;
      nonfinite = false;
      for (unsigned long long base = r_lo; base < r_hi; base += THREADS * 4ull) {
        const unsigned long long i0 = base + threadIdx.x * 4ull;
        uint32_t bits[4] = {0, 0, 0, 0};
        const int cnt = (i0 < r_hi) ? src.load_vals4(i0, p.n, bits) : 0;
        unsigned int fz = 0, fn = 0;
  #pragma unroll
        for (int e = 0; e < 4; ++e) {
          if (e < cnt) {
            if ((bits[e] & 0x7FFFFFFFu) != 0) fn |= 1u << e; else fz |= 1u << e;
          }
        }
        unsigned int z_total, keep_total;
        unsigned long long zrank = zeros_seen + block_excl_scan(__popc(fz), z_total, sh);
        unsigned int f = fn;
  #pragma unroll
        for (int e = 0; e < 4; ++e) {
          if (fz & (1u << e)) {
            if (zrank < allowed) f |= 1u << e;
            ++zrank;
          }
        }
        unsigned int pos = E + block_excl_scan(__popc(f), keep_total, sh);
  #pragma unroll
        for (int e = 0; e < 4; ++e) {
          if (f & (1u << e)) {
            const uint32_t key = bits[e] & 0x7FFFFFFFu;
            put_entry(pos, (uint32_t)(i0 + e), bits[e]);
            nonfinite |= key >= kInfKey;
            atomicAdd(&sh.hist[key >> digit_shift(0)], 1u);
            ++pos;
          }
        }
        zeros_seen += z_total;
        E += keep_total;
      }
      if (nonfinite) set_status(&p.ctl->status, NSML_ERR_NONFINITE);
      unsigned long long* totals2 = p.block_counts + 3 * kMaxFinalizeBlocks;
      if (threadIdx.x == 0) totals2[blk] = E;
      flush_hist<kMaxBins>(sh, p.hist + 3 * kMaxBins);
      if (!grid_barrier<CLUSTER>(p.ctl, ++barriers * G, sh)) return;
      unsigned long long part = 0;
      for (unsigned int b = threadIdx.x; b < G; b += THREADS) part += __ldcg(totals2 + b);
      if (block_sum(part, sh) < p.k) {  // cannot happen: the rebuilt list holds at least k entries
        if (threadIdx.x == 0) set_status(&p.ctl->status, NSML_ERR_INTERNAL);
        return;
      }
      ghist0 = p.hist + 3 * kMaxBins;
    }
  }
  __syncthreads();  // the block's array (shared copy and global) is complete

  // ---------------- phase 1: resolve digit 0, histogram of digit 1 ----------------
  resolve_digit<kMaxBins>(ghist0, (unsigned int)p.k, sh);
  const unsigned int d0 = sh.out[0];
  unsigned int rem = sh.out[1];
  for (int b = threadIdx.x; b < kMaxBins; b += THREADS) sh.hist[b] = 0;
  __syncthreads();
  for_each_key([&](uint32_t key) {
    if ((key >> 19) == d0) atomicAdd(&sh.hist[(key >> 7) & 0xFFFu], 1u);
  });
  flush_hist<kMaxBins>(sh, p.hist + 1 * kMaxBins);
  if (!grid_barrier<CLUSTER>(p.ctl, ++barriers * G, sh)) return;

  // ---------------- phase 2: resolve digit 1, histogram of digit 2 ----------------
  resolve_digit<kMaxBins>(p.hist + 1 * kMaxBins, rem, sh);
  const unsigned int prefix24 = (d0 << 12) | sh.out[0];
  rem = sh.out[1];
  __syncthreads();
  for (int b = threadIdx.x; b < 128; b += THREADS) sh.hist[b] = 0;
  __syncthreads();
  for_each_key([&](uint32_t key) {
    if ((key >> 7) == prefix24) atomicAdd(&sh.hist[key & 0x7Fu], 1u);
  });
  flush_hist<128>(sh, p.hist + 2 * kMaxBins);
  if (!grid_barrier<CLUSTER>(p.ctl, ++barriers * G, sh)) return;

  // ---------------- phase 3: T and r; count own keys > T and == T ----------------
  resolve_digit<128>(p.hist + 2 * kMaxBins, rem, sh);
  const uint32_t T = (prefix24 << 7) | sh.out[0];
  const unsigned long long r = sh.out[1];  // ties (key == T) to keep, lowest index first
  // Each warp owns two contiguous runs of the block's candidates: its slice of those cached in shared
  // memory and its slice of the rest (so that the slow loads of uncached values are spread over all
  // warps).  Here the keys > T and == T of each run are counted; the run totals stay in shared memory for
  // the write phase and their sum is the block's count.
  constexpr int NW = THREADS / 32;
  const int warp = threadIdx.x >> 5;
  const unsigned int lt = (1u << lane) - 1u;
  const unsigned int cached = min(E, (unsigned int)CACHE);
  unsigned int run_lo[2], run_hi[2];
  {
    const unsigned int per_a = ((cached + NW - 1) / NW + 31) / 32 * 32;
    const unsigned int per_b = ((E - cached + NW - 1) / NW + 31) / 32 * 32;
    run_lo[0] = min(cached, warp * per_a);
    run_hi[0] = min(cached, run_lo[0] + per_a);
    run_lo[1] = min(E, cached + warp * per_b);
    run_hi[1] = min(E, run_lo[1] + per_b);
  }
  __syncthreads();  // sh.run may still be read from an earlier call
#pragma unroll
  for (int q = 0; q < 2; ++q) {
    unsigned int wa = 0, wc = 0;
    for (unsigned int j0 = run_lo[q]; j0 < run_hi[q]; j0 += 128) {  // four rounds of 32, their loads issued together
      uint32_t key[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const unsigned int j = j0 + u * 32 + lane;
        key[u] = (j < run_hi[q]) ? (entry_val(j) & 0x7FFFFFFFu) : 0u;
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const bool live = j0 + u * 32 + lane < run_hi[q];
        wa += __popc(__ballot_sync(0xFFFFFFFFu, live && key[u] > T));
        wc += __popc(__ballot_sync(0xFFFFFFFFu, live && key[u] == T));
      }
    }
    if (lane == 0) sh.run[q * NW + warp] = ((unsigned long long)wa << 32) | wc;
  }
  __syncthreads();
  unsigned long long* ac_counts = p.block_counts + 1 * kMaxFinalizeBlocks;
  if (threadIdx.x == 0) {
    unsigned long long block_a = 0, block_c = 0;
    for (int w = 0; w < 2 * NW; ++w) {
      block_a += sh.run[w] >> 32;
      block_c += sh.run[w] & 0xFFFFFFFFull;
    }
    ac_counts[blk] = (block_a << 32) | block_c;
  }
  if (!grid_barrier<CLUSTER>(p.ctl, ++barriers * G, sh)) return;

  // ---------------- phase 4: write the survivors in index order ----------------
  unsigned long long a_before = 0, c_before = 0, a_all = 0, c_all = 0;
  for (unsigned int b = threadIdx.x; b < G; b += THREADS) {
    const unsigned long long w = __ldcg(ac_counts + b);
    a_all += w >> 32;
    c_all += w & 0xFFFFFFFFull;
    if (b < blk) {
      a_before += w >> 32;
      c_before += w & 0xFFFFFFFFull;
    }
  }
  a_before = block_sum(a_before, sh);
  c_before = block_sum(c_before, sh);
  a_all = block_sum(a_all, sh);
  c_all = block_sum(c_all, sh);
  if (a_all + min(c_all, r) != p.k) {
    if (threadIdx.x == 0) set_status(&p.ctl->status, NSML_ERR_INTERNAL);
    return;
  }
  uint32_t* out_idx = reinterpret_cast<uint32_t*>(p.payload + p.P.idx_off);
  {
    // ranks by ballot on top of the run totals counted in phase 3, coalesced writes
#pragma unroll
    for (int q = 0; q < 2; ++q) {
      unsigned long long a_here = a_before, c_here = c_before;
      for (int w = 0; w < q * NW + warp; ++w) {  // runs in index order: every warp's cached run, then the others
        a_here += sh.run[w] >> 32;
        c_here += sh.run[w] & 0xFFFFFFFFull;
      }
      for (unsigned int j0 = run_lo[q]; j0 < run_hi[q]; j0 += 128) {
        uint32_t bits[4], idx[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const unsigned int j = j0 + u * 32 + lane;
          bits[u] = (j < run_hi[q]) ? entry_val(j) : 0u;
          idx[u] = (j < run_hi[q]) ? my_idx[j] : 0u;  // coalesced; read whether or not the entry survives
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const bool live = j0 + u * 32 + lane < run_hi[q];
          const uint32_t key = bits[u] & 0x7FFFFFFFu;
          const bool a = live && key > T;
          const bool c = live && key == T;
          const unsigned int ba = __ballot_sync(0xFFFFFFFFu, a), bc = __ballot_sync(0xFFFFFFFFu, c);
          const unsigned long long a_mine = a_here + __popc(ba & lt), c_mine = c_here + __popc(bc & lt);
          if (a || (c && c_mine < r)) {
            const unsigned long long pos = a_mine + min(c_mine, r);
            out_idx[pos] = idx[u];
            put_value(p, pos, bits[u]);
          }
          a_here += __popc(ba);
          c_here += __popc(bc);
        }
      }
    }
  }
  // ---------------- phase 5: the header; int8: quantise ----------------
  if (blk == 0 && threadIdx.x == 0) write_header(p);
  if (p.bits != NSML_BITS_INT8) return;  // float32 and fp16 values are in the payload already
  if (!grid_barrier<CLUSTER>(p.ctl, ++barriers * G, sh)) return;
  quantize_all(p, sh);
}

}  // namespace nsml
