// Shared definitions for the libnsml device code (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <stdint.h>

#include "nsml.h"

namespace nsml {

// Radix digits of the 31-bit magnitude key, most significant first:
// bits 30..19 (8 exponent + 4 mantissa bits), bits 18..7, bits 6..0.
__host__ __device__ constexpr int digit_bits(int level) { return level == 2 ? 7 : 12; }
__host__ __device__ constexpr int digit_shift(int level) { return level == 0 ? 19 : (level == 1 ? 7 : 0); }
constexpr int kMaxBins = 4096;

constexpr int kCta = 256;          // threads per block in every streaming kernel
constexpr uint32_t kInfKey = 0x7F800000u;
constexpr int kStreamLoads = 4;                       // 16-byte loads a thread of a streaming kernel keeps in flight
constexpr int kStreamTile = kCta * 4 * kStreamLoads;  // elements a block of a streaming kernel takes per step

// Polls before a wait at a grid barrier gives up (each poll sleeps a little,
// so this is on the order of a second).
constexpr int kMaxPolls = 1 << 22;

// Control block at the start of a compress workspace.  Cleared (together with
// the histograms and counters that follow it) at the start of every call.
struct Ctl {
  int status;                 // first device-detected error (NSML_ERR_*), 0 = ok
  unsigned int lo;            // sampled lower bound of the threshold key: candidates are the keys >= max(lo, 1)
  unsigned int barrier;       // arrivals at the grid barriers of the cooperative kernel
  unsigned int shift;         // fine histogram: bin = min((key - lo) >> shift, kFineBins - 1)
  unsigned int exact;         // every fine bin below the last holds one representable key value
  unsigned int und_count;     // entries appended to the list of undecided candidates
  unsigned int fallback;      // the list stage gave up (too few candidates, a full table): select over the bucket
  unsigned int mark_done;     // blocks of the bucket pass that have finished
  unsigned int pick_done;     // blocks of the first list kernel that have finished
  unsigned int Tbin;          // fine bin that holds the k-th largest key
  unsigned int rem;           // rank of that key inside its bin, from the top
  unsigned int by_bin;        // the bin itself decides: above it = above T, in it = equal to T (exact && Tbin not the last)
  unsigned int T;             // listed case: the threshold key ...
  unsigned int limit;         // ... and the index up to which ties at T survive
  unsigned int ties_kept;     // by-bin case: keys equal to T that survive, lowest index first
};
static_assert(sizeof(Ctl) <= 256, "control block must fit its 256-byte slot");

constexpr int kSegElems = 512;            // bucket elements per ownership unit of the dense select
constexpr int kMaxFinalizeBlocks = 1024;  // upper bound on blocks of the cooperative kernels
constexpr int kFineBins = 2048;           // bins of the candidates' key histogram built by the bucket pass
constexpr int kFineStride = 32;            // words between two bins' counters: neighbouring bins, which are hot together, sit in different 128-byte lines
constexpr int kGroupElems = 4096;         // bucket elements per group; the bucket pass keeps a candidate count per group
constexpr int kPickGroups = 8;            // groups (32768 elements) a block of the list stage owns
constexpr int kPickElems = kPickGroups * kGroupElems;
constexpr int kStashPerBlock = kPickElems;      // values of one block's candidates the stash holds: room for every element
constexpr int kRoundElems = 128;          // bucket elements per round: 4 words (16 bytes) of the candidate bitmap
constexpr unsigned int kUndCap = 2048;    // undecided candidates (those in the threshold's fine bin) that can be listed

struct CompressLayout {  // byte offsets inside a compress workspace
  size_t hist;          // u32[4][kMaxBins]: digit histograms of the dense select
  size_t fine;          // u32[kFineBins * kFineStride]: candidates per fine key bin (one counter per 128-byte line)
  size_t group_count;   // u32[ceil(n / kGroupElems)]: candidates per group
  size_t qcount;        // u32[n / 4096 + 2]: survivors delivered so far per block of 1024 payload entries
  size_t zero_bytes;    // everything before this offset is cleared per call
  size_t block_counts;  // u64[4][kMaxFinalizeBlocks]: per-block counts exchanged at barriers (dense select)
  size_t und;           // uint2[kUndCap]: (value bits, index) of the undecided candidates
  size_t per_block;     // u32[6][ceil(n / kPickElems)]: list stage, per block: candidates, above the bin, in the bin,
                        //   listed survivors, survivors before the block, in-bin entries before the block
  size_t bitmap;        // u32[4 * ceil(n / kRoundElems)]: bit (i & 31) of word i >> 5 set = element i is a candidate
  size_t raw_val;       // f32[n]: survivor values before quantisation (list strategy: at most n / 4 of them) ...
  size_t stash;         // ... list strategy: u32[ceil(n / kPickElems) * kPickElems]: values of each block's candidates
  size_t total;
};

__host__ __device__ inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

inline CompressLayout compress_layout(int64_t n) {
  CompressLayout L;
  const size_t groups = ((size_t)n + kGroupElems - 1) / kGroupElems;
  const size_t rounds = ((size_t)n + kRoundElems - 1) / kRoundElems;
  const size_t pick_blocks = ((size_t)n + kPickElems - 1) / kPickElems;
  L.hist = 256;
  L.fine = L.hist + 4 * kMaxBins * sizeof(unsigned int);
  L.group_count = L.fine + (size_t)kFineBins * kFineStride * sizeof(unsigned int);
  L.qcount = L.group_count + align_up(groups * 4, 256);
  L.zero_bytes = L.qcount + align_up(((size_t)n / 4096 + 2) * 4, 256);
  L.block_counts = L.zero_bytes;
  L.und = L.block_counts + 4 * kMaxFinalizeBlocks * 8;
  L.per_block = L.und + (size_t)kUndCap * 8;
  L.bitmap = L.per_block + align_up(6 * pick_blocks * 4, 256);
  L.raw_val = L.bitmap + align_up(rounds * 16, 256);
  // the dense select keeps up to n raw values; the list strategy n / 4 raw values and the stash behind them
  L.stash = L.raw_val + align_up(((size_t)n / 4 + 1024) * 4, 256);
  L.total = L.stash + pick_blocks * (size_t)kStashPerBlock * 4;
  if (L.total < L.raw_val + align_up((size_t)n * 4, 256)) L.total = L.raw_val + align_up((size_t)n * 4, 256);
  return L;
}

struct PayloadLayout {
  int64_t k;
  size_t idx_off, val_off, scale_off, nblocks, total;
};

inline PayloadLayout payload_layout(int64_t k, int bits) {
  PayloadLayout P;
  P.k = k;
  P.idx_off = sizeof(nsml_payload_header);
  P.val_off = P.idx_off + align_up((size_t)k * 4, 16);
  if (bits == NSML_BITS_INT8) {
    P.nblocks = (size_t)((k + NSML_QBLOCK - 1) / NSML_QBLOCK);
    P.scale_off = P.val_off + align_up((size_t)k, 16);
    P.total = P.scale_off + align_up(P.nblocks * 4, 16);
  } else {  // fp16: 2 bytes per value; float32 as is: 4
    P.nblocks = 0;
    P.scale_off = 0;
    P.total = P.val_off + align_up((size_t)k * (bits == NSML_BITS_FP32 ? 4 : 2), 16);
  }
  return P;
}

__device__ __forceinline__ void set_status(int* status, int code) { atomicCAS(status, 0, code); }

// ------------------------------------------------------------------------
// Element sources.  load_vals4 returns the float32 bit patterns of elements
// i0..i0+3 (i0 a multiple of 4) and how many of them exist (0..4); missing
// ones read as 0.  Pruned elements (mask bit set) read as +0.0.
// ------------------------------------------------------------------------
template <int DTYPE>
struct BucketSrc {
  const void* grad;
  const uint32_t* mask;  // may be null

  __device__ __forceinline__ int load_vals4(unsigned long long i0, unsigned long long count, uint32_t (&bits)[4]) const {
    int cnt;
    if (i0 + 4 <= count) {
      if (DTYPE == NSML_F32) {
        const uint4 v = __ldcs(reinterpret_cast<const uint4*>(static_cast<const uint32_t*>(grad) + i0));
        bits[0] = v.x; bits[1] = v.y; bits[2] = v.z; bits[3] = v.w;
      } else {
        const uint2 v = __ldcs(reinterpret_cast<const uint2*>(static_cast<const uint16_t*>(grad) + i0));
        bits[0] = v.x << 16; bits[1] = v.x & 0xFFFF0000u;
        bits[2] = v.y << 16; bits[3] = v.y & 0xFFFF0000u;
      }
      cnt = 4;
    } else {
      cnt = (i0 < count) ? (int)(count - i0) : 0;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        bits[e] = 0;
        if (e < cnt) {
          if (DTYPE == NSML_F32) bits[e] = static_cast<const uint32_t*>(grad)[i0 + e];
          else bits[e] = (uint32_t)static_cast<const uint16_t*>(grad)[i0 + e] << 16;
        }
      }
    }
    if (mask != nullptr && cnt > 0) {
      const uint32_t m = (mask[i0 >> 5] >> (unsigned)(i0 & 31)) & 0xFu;
#pragma unroll
      for (int e = 0; e < 4; ++e)
        if (m & (1u << e)) bits[e] = 0;
    }
    return cnt;
  }

  // elements i0..i0+3 all exist (no bounds checks)
  __device__ __forceinline__ void load_full4(unsigned long long i0, uint32_t (&bits)[4]) const {
    if (DTYPE == NSML_F32) {
      const uint4 v = __ldcs(reinterpret_cast<const uint4*>(static_cast<const uint32_t*>(grad) + i0));
      bits[0] = v.x; bits[1] = v.y; bits[2] = v.z; bits[3] = v.w;
    } else {
      const uint2 v = __ldcs(reinterpret_cast<const uint2*>(static_cast<const uint16_t*>(grad) + i0));
      bits[0] = v.x << 16; bits[1] = v.x & 0xFFFF0000u;
      bits[2] = v.y << 16; bits[3] = v.y & 0xFFFF0000u;
    }
    if (mask != nullptr) {
      const uint32_t m = (mask[i0 >> 5] >> (unsigned)(i0 & 31)) & 0xFu;
#pragma unroll
      for (int e = 0; e < 4; ++e)
        if (m & (1u << e)) bits[e] = 0;
    }
  }

  // elements i0..i0+3 as stored (all exist; no pruning mask applied), and the mask's four flags for them
  __device__ __forceinline__ void load_raw4(unsigned long long i0, uint32_t (&bits)[4]) const {
    if (DTYPE == NSML_F32) {
      const uint4 v = __ldcs(reinterpret_cast<const uint4*>(static_cast<const uint32_t*>(grad) + i0));
      bits[0] = v.x; bits[1] = v.y; bits[2] = v.z; bits[3] = v.w;
    } else {
      const uint2 v = __ldcs(reinterpret_cast<const uint2*>(static_cast<const uint16_t*>(grad) + i0));
      bits[0] = v.x << 16; bits[1] = v.x & 0xFFFF0000u;
      bits[2] = v.y << 16; bits[3] = v.y & 0xFFFF0000u;
    }
  }
  __device__ __forceinline__ unsigned int pruned4(unsigned long long i0) const {
    return mask != nullptr ? (mask[i0 >> 5] >> (unsigned)(i0 & 31)) & 0xFu : 0u;
  }

  // element i as stored (no pruning mask applied), and whether the mask prunes it
  __device__ __forceinline__ uint32_t raw1(unsigned long long i) const {
    if (DTYPE == NSML_F32) return static_cast<const uint32_t*>(grad)[i];
    return (uint32_t)static_cast<const uint16_t*>(grad)[i] << 16;
  }
  __device__ __forceinline__ bool pruned(unsigned long long i) const {
    return mask != nullptr && ((mask[i >> 5] >> (unsigned)(i & 31)) & 1u);
  }

  __device__ __forceinline__ uint32_t load1(unsigned long long i) const {
    if (mask != nullptr && ((mask[i >> 5] >> (unsigned)(i & 31)) & 1u)) return 0;
    if (DTYPE == NSML_F32) return static_cast<const uint32_t*>(grad)[i];
    return (uint32_t)static_cast<const uint16_t*>(grad)[i] << 16;
  }
};

}  // namespace nsml
