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

// Polls before a wait at a grid barrier gives up (each poll sleeps a little,
// so this is on the order of a second).
constexpr int kMaxPolls = 1 << 22;

// Control block at the start of a compress workspace.  Cleared (together with
// the histograms that follow it) at the start of every call.
struct Ctl {
  int status;                 // first device-detected error (NSML_ERR_*), 0 = ok
  unsigned int lo;            // sampled lower bound of the threshold key
  unsigned int barrier;       // arrivals at the finalize kernel's grid barriers
  unsigned int pad;
};
static_assert(sizeof(Ctl) <= 256, "control block must fit its 256-byte slot");

constexpr int kSegElems = 512;            // bucket elements per candidate-list segment (4 rounds of 128)
constexpr int kGroupSegs = 64;            // segments per group; the bucket pass keeps a candidate count per group
constexpr int kMaxFinalizeBlocks = 1024;  // upper bound on blocks of the finalize kernel

struct CompressLayout {  // byte offsets inside a compress workspace
  size_t hist;          // u32[4][kMaxBins]: digit histograms (levels 0..2, level 0 again after a rebuild)
  size_t group_count;   // u32[ceil(segments / kGroupSegs)]: candidates per group of segments
  size_t zero_bytes;    // everything before this offset is cleared per call 
  size_t block_counts;  // u64[4][kMaxFinalizeBlocks]: per-block counts exchanged at barriers
  size_t seg_count;     // u16[ceil(n / kSegElems)]: entries per segment
  size_t seg_off;       // u16[n]: segmented candidate list (bucket pass output), a candidate's offset inside its segment; segment s starts at s * kSegElems
  size_t seg_val;       // u32[n] (float32 bit patterns)
  size_t list_idx;      // u32[n]: the same candidates, contiguous per finalize block
  size_t list_val;      // u32[n]
  size_t raw_val;       // f32[n]: survivor values before quantisation (the same memory as seg_val)
  size_t total;
};

__host__ __device__ inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

inline CompressLayout compress_layout(int64_t n) {
  CompressLayout L;
  const size_t npad = align_up((size_t)n, kSegElems);
  const size_t segs = npad / kSegElems;
  L.hist = 256;
  L.group_count = L.hist + 4 * kMaxBins * sizeof(unsigned int);
  L.zero_bytes = L.group_count + align_up(((segs + kGroupSegs - 1) / kGroupSegs) * 4, 256);
  L.block_counts = L.zero_bytes;
  L.seg_count = L.block_counts + 4 * kMaxFinalizeBlocks * 8;
  L.seg_off = L.seg_count + align_up(segs * 2, 256);
  L.seg_val = L.seg_off + npad * 2;
  L.list_idx = L.seg_val + npad * 4;
  L.list_val = L.list_idx + npad * 4;
  // raw_val shares the memory of seg_val: the segmented list is dead once k_gather has copied it, the
  // survivors' raw values are written after that (list strategy), and the dense strategy has no list at all
  L.raw_val = L.seg_val;
  L.total = L.list_val + npad * 4;
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
