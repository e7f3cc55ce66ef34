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
constexpr int kTile = 4096;        // elements per compaction tile (16 per thread)
constexpr uint32_t kInfKey = 0x7F800000u;

// Tile-state word of the chained scan: [63:62] flag, [61:31] count A, [30:0] count C.
constexpr unsigned long long kFlagAggregate = 1ull << 62;  // this tile's own counts
constexpr unsigned long long kFlagPrefix = 2ull << 62;     // inclusive prefix up to this tile
constexpr unsigned long long kFlagAbort = 3ull << 62;      // a predecessor gave up
constexpr unsigned long long kFlagMask = 3ull << 62;
constexpr unsigned long long kCountMask = (1ull << 31) - 1;

// Polls of one predecessor window before a look-back gives up (each poll sleeps
// a little, so this is on the order of a second).
constexpr int kMaxPolls = 1 << 21;

// Control block at the start of a compress workspace.  Zeroed (together with
// the histograms and tile states that follow it) at the start of every call.
struct Ctl {
  int status;                     // first device-detected error (NSML_ERR_*), 0 = ok
  unsigned int ticket_bucket;     // next tile of the bucket compaction
  unsigned int ticket_list;       // next tile of the list compaction
  unsigned int done[3];           // blocks that finished histogram level 0..2
  unsigned int exact;             // 1: threshold key and tie budget are final
  unsigned int prefix;            // resolved high bits of the threshold key
  unsigned int lo, hi;            // class A: key >= hi; class C: lo <= key < hi
  unsigned long long r;           // class-C entries taken, lowest index first
  unsigned long long k_rem;       // survivors still to find among keys matching prefix
  unsigned long long zero_count;  // keys equal to 0 in the bucket
  unsigned long long list_count;  // entries the bucket compaction wrote
  unsigned long long out_count;   // entries the list compaction wrote (must equal k)
};
static_assert(sizeof(Ctl) <= 256, "control block must fit its 256-byte slot");

struct CompressLayout {  // byte offsets inside a compress workspace
  size_t hist;        // u32[3][kMaxBins]
  size_t state_bucket;  // u64[tiles]
  size_t state_list;    // u64[tiles]
  size_t zero_bytes;    // everything before this offset is cleared per call
  size_t list_idx;      // u32[n]
  size_t list_val;      // u32[n] (float32 bit patterns)
  size_t raw_val;       // f32[n]
  size_t total;
};

__host__ __device__ inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

inline CompressLayout compress_layout(int64_t n) {
  CompressLayout L;
  size_t tiles = (size_t)((n + kTile - 1) / kTile);
  size_t npad = align_up((size_t)n, 64);
  L.hist = 256;
  L.state_bucket = L.hist + 3 * kMaxBins * sizeof(unsigned int);
  L.state_list = L.state_bucket + align_up(tiles * 8, 256);
  L.zero_bytes = L.state_list + align_up(tiles * 8, 256);
  L.list_idx = L.zero_bytes;
  L.list_val = L.list_idx + npad * 4;
  L.raw_val = L.list_val + npad * 4;
  L.total = L.raw_val + npad * 4;
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
  } else {
    P.nblocks = 0;
    P.scale_off = 0;
    P.total = P.val_off + align_up((size_t)k * 2, 16);
  }
  return P;
}

__device__ __forceinline__ void set_status(int* status, int code) { atomicCAS(status, 0, code); }

// ------------------------------------------------------------------------
// Element sources.  load4 returns the float32 bit patterns and indices of
// elements i0..i0+3 (i0 a multiple of 4); lanes beyond `count` report
// valid = false.  Pruned elements (mask bit set) read as +0.0.
// ------------------------------------------------------------------------
struct Quad {
  uint32_t bits[4];
  uint32_t idx[4];
  uint32_t valid;  // bit q set: element q exists
};

template <int DTYPE>
struct BucketSrc {
  const void* grad;
  const uint32_t* mask;  // may be null

  __device__ __forceinline__ Quad load4(unsigned long long i0, unsigned long long count) const {
    Quad q;
    q.valid = 0;
    if (i0 + 4 <= count) {
      if (DTYPE == NSML_F32) {
        uint4 v = *reinterpret_cast<const uint4*>(static_cast<const uint32_t*>(grad) + i0);
        q.bits[0] = v.x; q.bits[1] = v.y; q.bits[2] = v.z; q.bits[3] = v.w;
      } else {
        uint2 v = *reinterpret_cast<const uint2*>(static_cast<const uint16_t*>(grad) + i0);
        q.bits[0] = v.x << 16; q.bits[1] = v.x & 0xFFFF0000u;
        q.bits[2] = v.y << 16; q.bits[3] = v.y & 0xFFFF0000u;
      }
      q.valid = 0xF;
    } else {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        q.bits[e] = 0;
        if (i0 + e < count) {
          q.valid |= 1u << e;
          if (DTYPE == NSML_F32) q.bits[e] = static_cast<const uint32_t*>(grad)[i0 + e];
          else q.bits[e] = (uint32_t)static_cast<const uint16_t*>(grad)[i0 + e] << 16;
        }
      }
    }
    if (mask != nullptr && q.valid) {
      uint32_t m = (mask[i0 >> 5] >> (unsigned)(i0 & 31)) & 0xFu;
#pragma unroll
      for (int e = 0; e < 4; ++e)
        if (m & (1u << e)) q.bits[e] = 0;
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) q.idx[e] = (uint32_t)(i0 + e);
    return q;
  }
};

struct ListSrc {
  const uint32_t* idx;
  const uint32_t* val;

  __device__ __forceinline__ Quad load4(unsigned long long i0, unsigned long long count) const {
    Quad q;
    q.valid = 0;
    if (i0 + 4 <= count) {
      uint4 a = *reinterpret_cast<const uint4*>(idx + i0);
      uint4 b = *reinterpret_cast<const uint4*>(val + i0);
      q.idx[0] = a.x; q.idx[1] = a.y; q.idx[2] = a.z; q.idx[3] = a.w;
      q.bits[0] = b.x; q.bits[1] = b.y; q.bits[2] = b.z; q.bits[3] = b.w;
      q.valid = 0xF;
    } else {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        q.bits[e] = 0;
        q.idx[e] = 0;
        if (i0 + e < count) {
          q.valid |= 1u << e;
          q.idx[e] = idx[i0 + e];
          q.bits[e] = val[i0 + e];
        }
      }
    }
    return q;
  }
};

}  // namespace nsml
