// Bucket -> segmented candidate list: the one full pass over the bucket
// (Alg. 2 Steps 2-3: pruned gradients read as zero; everything whose magnitude
// is below the sampled lower bound is dropped here, in one streaming read).
//
// The bucket is cut into segments of kSegElems elements.  A warp takes one
// segment at a time and appends what it keeps (every key >= lo, lo >= 1) to
// the segment's own slots of the list, [s * kSegElems, s * kSegElems + count),
// so nothing can overflow, nothing is allocated and no warp ever waits for
// another: there is no block or grid synchronisation in this kernel.
// Segments in increasing order are in index order.
//
// Blocks walk the bucket block-cyclically (block b takes segments 8b..8b+7,
// then 8(b+G).., ...), so at any moment the whole grid reads one compact
// window of the bucket, which is what DRAM row buffers like.  Every lane
// keeps its part of the warp's next segment in flight: in registers (16-byte
// loads issued a segment or two ahead), or, when a residual is streamed
// beside the gradient, with asynchronous copies into a private
// shared-memory slot, which a lane reads back only itself, so neither
// buffer needs any synchronisation.
#pragma once

#include "nsml_common.cuh"

namespace nsml {

// dynamic shared memory of the bucket pass with local accumulation: the residual's double buffers
// (a warp's segment of the residual: kSegElems float32, two of them per warp)
constexpr size_t kCompactFeedbackSmem = (size_t)(kCta / 32) * 2 * kSegElems * 4;

// Appends the kept elements of one round of 32 * EPL elements.  `f` holds this lane's keep flags (bit e =
// element lane*EPL+e of the round).  Returns the round's total.
template <int EPL>
__device__ __forceinline__ unsigned int append_round(unsigned int f, const uint32_t (&bits)[EPL], unsigned int first_offset,
                                                     unsigned long long out_base, unsigned short* __restrict__ seg_off,
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
    for (int e = 0; e < EPL; ++e) {
      if (f & (1u << e)) {
        seg_off[pos] = (unsigned short)(first_offset + lane * EPL + e);
        seg_val[pos] = bits[e];
        ++pos;
      }
    }
  }
  return total;
}

// ---- per-lane asynchronous copies (global -> shared) ----
template <int BYTES>
__device__ __forceinline__ void cp_async_lane(void* smem_dst, const void* gsrc) {
  const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
  if (BYTES == 16) asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(gsrc) : "memory");
  else asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(d), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int PENDING>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(PENDING) : "memory"); }

// |v| >= t on floats equals key >= lo for finite v; written as !(|v| < t) so
// that NaN is kept too (the finalize kernel reports non-finite candidates).
template <int EPL>
__device__ __forceinline__ unsigned int keep_flags(const uint32_t (&bits)[EPL], float t) {
  unsigned int f = 0;
#pragma unroll
  for (int e = 0; e < EPL; ++e) f |= (unsigned)(!(fabsf(__uint_as_float(bits[e])) < t)) << e;
  return f;
}

// One segment's worth of 16-byte loads of a lane, unpacked: float32 as is, bfloat16 widened to float32 bit patterns.
template <int DTYPE, int EPL>
__device__ __forceinline__ void unpack16(const uint4& v, uint32_t (&bits)[EPL]) {
  if (DTYPE == NSML_F32) {
    bits[0] = v.x; bits[1] = v.y; bits[2] = v.z; bits[3] = v.w;
  } else {
    bits[0] = v.x << 16; bits[1] = v.x & 0xFFFF0000u;
    bits[2] = v.y << 16; bits[3] = v.y & 0xFFFF0000u;
    bits[4 % EPL] = v.z << 16; bits[5 % EPL] = v.z & 0xFFFF0000u;
    bits[6 % EPL] = v.w << 16; bits[7 % EPL] = v.w & 0xFFFF0000u;
  }
}

// The bucket pass without a residual: NOT a persistent kernel.  A warp takes 2 KB of the bucket (one float32
// segment, two bfloat16 segments), issues all of its 16-byte loads at once and is done; a block is eight
// warps on 16 consecutive KB, and the hardware's block scheduler, which hands out blocks in order, keeps the
// grid on one compact, moving window of the bucket.  Measured on a 100 MB float32 bucket whose candidates
// crowd into a few tensors: 19.0 us, against 19.9 us for persistent blocks that prefetch the next segment into
// registers, 21.9 us for a shared-memory ring of asynchronous copies and 18.6 us for a plain read of the
// bucket; blocks that own 2, 4, 8 consecutive 16 KB steps take 20.5, 23.4, 29.4 us (the wider the window of
// addresses in flight, the slower).  Short-lived blocks also share the SMs gracefully with other streams'
// kernels, where a grid of persistent blocks that does not fit at once runs a second wave.  MASKED: a pruning
// mask is applied (a segment's 16 mask words are fetched by lanes 0-15 with the data and handed out by shuffle).
template <int DTYPE>
__host__ __device__ constexpr int compact_segs_per_warp() { return DTYPE == NSML_F32 ? 1 : 2; }

template <int DTYPE, bool MASKED>
__device__ __forceinline__ void compact_plain(const BucketSrc<DTYPE>& src, unsigned long long n, const Ctl* ctl,
                                              unsigned short* __restrict__ seg_off, uint32_t* __restrict__ seg_val,
                                              unsigned short* __restrict__ seg_count, unsigned int* __restrict__ group_count) {
  constexpr int ESIZE = (DTYPE == NSML_F32) ? 4 : 2;
  constexpr int EPL = 16 / ESIZE;                 // elements a lane takes per round: 16 bytes' worth
  constexpr int ROUND = 32 * EPL;                 // elements a warp handles per step
  constexpr int ROUNDS = kSegElems / ROUND;       // steps per segment: 4 or 2
  constexpr int SEGS = compact_segs_per_warp<DTYPE>();
  constexpr int kSegMaskWords = kSegElems / 32;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const unsigned long long nseg = (n + kSegElems - 1) / kSegElems;
  const unsigned long long nseg_full = n / kSegElems;  // segments that need no bounds checks
  const unsigned long long first = ((unsigned long long)blockIdx.x * (kCta / 32) + w) * SEGS;
  if (first >= nseg) return;
  const uint4* g = reinterpret_cast<const uint4*>(src.grad) + lane;  // round r of segment s: g[(s * ROUNDS + r) * 32]
  uint4 q[SEGS][ROUNDS];
  uint32_t mw[SEGS];
#pragma unroll
  for (int s = 0; s < SEGS; ++s) {
    mw[s] = 0;
    if (first + s < nseg_full) {
#pragma unroll
      for (int r = 0; r < ROUNDS; ++r) q[s][r] = __ldcs(g + ((first + s) * ROUNDS + r) * 32);
      if (MASKED && lane < kSegMaskWords) mw[s] = __ldg(src.mask + (first + s) * kSegMaskWords + lane);
    }
  }
  // Zeros are never candidates here; if they are needed (fewer than k non-zero
  // keys) the list comes out short and the finalize kernel's slow path adds them.
  const float t = __uint_as_float(max(ctl->lo, 1u));
#pragma unroll
  for (int s = 0; s < SEGS; ++s) {
    const unsigned long long seg = first + s;
    if (seg >= nseg) break;
    const unsigned long long seg_base = seg * kSegElems;
    unsigned int kept = 0;
#pragma unroll
    for (int r = 0; r < ROUNDS; ++r) {
      uint32_t bits[EPL];
      if (seg < nseg_full) {
        unpack16<DTYPE, EPL>(q[s][r], bits);
        if (MASKED) {
          // this lane's EPL mask bits inside the round's ROUND / 32 words
          const uint32_t word = __shfl_sync(0xFFFFFFFFu, mw[s], r * (ROUND / 32) + lane * EPL / 32);
          const uint32_t m = (word >> (unsigned)((lane * EPL) & 31)) & ((1u << EPL) - 1u);
#pragma unroll
          for (int e = 0; e < EPL; ++e)
            if (m & (1u << e)) bits[e] = 0;
        }
      } else {
        // the bucket's ragged last segment: plain loads, missing elements read as 0 and are never kept
        // (load_vals4 applies the mask)
#pragma unroll
        for (int qq = 0; qq < EPL / 4; ++qq) {
          uint32_t four[4];
          src.load_vals4(seg_base + r * ROUND + lane * EPL + qq * 4, n, four);
#pragma unroll
          for (int e = 0; e < 4; ++e) bits[qq * 4 + e] = four[e];
        }
      }
      const unsigned int f = keep_flags<EPL>(bits, t);
      if (!__any_sync(0xFFFFFFFFu, f != 0)) continue;
      kept += append_round<EPL>(f, bits, (unsigned int)(r * ROUND), seg_base + kept, seg_off, seg_val);
    }
    if (lane == 0) {
      seg_count[seg] = (unsigned short)kept;
      if (kept) atomicAdd(group_count + seg / kGroupSegs, kept);  // result unused: a fire-and-forget reduction
    }
  }
}

// FEEDBACK: the bucket that is compressed is gradient + residual (Section 4.2 Step 3, local accumulation of
// the filtered gradients).  The residual is streamed beside the gradient, the sum (one float32 add per
// element) is written back over the residual and is what the candidates are taken from; the pruning mask
// zeroes a key, not the stored sum.  Here every lane keeps its part of the warp's next segment (gradient and
// residual) in flight with asynchronous copies into a private shared-memory slot: a lane reads back only what
// it copied itself, so the double buffer needs no synchronisation.
template <int DTYPE, bool FEEDBACK = false, bool MASKED = true>
__global__ void __launch_bounds__(kCta)
k_compact_bucket(BucketSrc<DTYPE> src, float* __restrict__ residual, unsigned long long n, Ctl* ctl,
                 unsigned short* __restrict__ seg_off, uint32_t* __restrict__ seg_val, unsigned short* __restrict__ seg_count,
                 unsigned int* __restrict__ group_count) {
  if (!FEEDBACK) {
    compact_plain<DTYPE, MASKED>(src, n, ctl, seg_off, seg_val, seg_count, group_count);
    return;
  }
  constexpr int ESIZE = (DTYPE == NSML_F32) ? 4 : 2;
  constexpr int EPL = 4;                          // beside the residual (float32, 16 bytes per 4 elements) a lane takes 4 elements
  constexpr int ROUND = 32 * EPL;                 // elements a warp handles per step
  constexpr int ROUNDS = kSegElems / ROUND;       // steps per segment
  constexpr int LANE_BYTES = EPL * ESIZE;         // 16, or 8 (bfloat16)
  constexpr int BUF_BYTES = kSegElems * ESIZE;    // one segment of one warp
  constexpr int RBUF_BYTES = kSegElems * 4;       // the same segment of the residual
  __shared__ __align__(16) unsigned char s_fifo[FEEDBACK ? (kCta / 32) * 2 * BUF_BYTES : 16];
  extern __shared__ __align__(16) unsigned char s_rfifo[];  // (kCta / 32) * 2 * RBUF_BYTES bytes
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  unsigned char* fifo = s_fifo + (FEEDBACK ? (size_t)w * 2 * BUF_BYTES + lane * LANE_BYTES : 0);  // round r of buffer b at + (b*ROUNDS + r)*32*LANE_BYTES
  unsigned char* rfifo = s_rfifo + (size_t)w * 2 * RBUF_BYTES + lane * 16;       // the same for the residual: + (b*ROUNDS + r)*32*16

  const unsigned long long nseg = (n + kSegElems - 1) / kSegElems;
  const unsigned long long nseg_full = n / kSegElems;  // segments that need no bounds checks
  const unsigned long long step = (unsigned long long)gridDim.x * (kCta / 32);
  const unsigned char* g = static_cast<const unsigned char*>(src.grad) + (size_t)lane * LANE_BYTES;

  // asynchronous copies of one whole segment into buffer b (nothing for the ragged last segment, which is
  // read with plain loads); one commit group per segment, empty or not
  auto fetch = [&](unsigned long long s, int b) {
    if (s < nseg_full) {
#pragma unroll
      for (int r = 0; r < ROUNDS; ++r) {
        cp_async_lane<LANE_BYTES>(fifo + (b * ROUNDS + r) * 32 * LANE_BYTES, g + (s * kSegElems + r * ROUND) * ESIZE);
        cp_async_lane<16>(rfifo + (b * ROUNDS + r) * 32 * 16, residual + s * kSegElems + r * ROUND + lane * 4);
      }
    }
    cp_async_commit();
  };

  unsigned long long seg = (unsigned long long)blockIdx.x * (kCta / 32) + w;
  fetch(seg, 0);
  // The segment's 16 words of the pruning mask (64 bytes) are fetched by lanes 0-15 one segment ahead, like
  // the data, and handed to the lanes by shuffle.
  constexpr int kSegMaskWords = kSegElems / 32;
  uint32_t mask_words = 0, mask_words_next = 0;
  if (src.mask != nullptr && seg < nseg_full && lane < kSegMaskWords) mask_words = __ldg(src.mask + seg * kSegMaskWords + lane);
  // Zeros are never candidates here; if they are needed (fewer than k non-zero
  // keys) the list comes out short and the finalize kernel's slow path adds them.
  const float t = __uint_as_float(max(ctl->lo, 1u));
  int buf = 0;

  while (seg < nseg) {
    const unsigned long long next = seg + step;
    fetch(next, buf ^ 1);
    if (src.mask != nullptr && next < nseg_full && lane < kSegMaskWords)
      mask_words_next = __ldg(src.mask + next * kSegMaskWords + lane);
    cp_async_wait<1>();  // this segment's copies have landed; the next segment's stay in flight

    const unsigned long long seg_base = seg * kSegElems;
    unsigned int kept = 0;
#pragma unroll
    for (int r = 0; r < ROUNDS; ++r) {
      uint32_t bits[EPL];
      if (seg < nseg_full) {
        const unsigned char* slot = fifo + (buf * ROUNDS + r) * 32 * LANE_BYTES;
        if (DTYPE == NSML_F32) {
          const uint4 v = *reinterpret_cast<const uint4*>(slot);
          bits[0] = v.x; bits[1] = v.y; bits[2] = v.z; bits[3] = v.w;
        } else {
          const uint2 v = *reinterpret_cast<const uint2*>(slot);
          bits[0] = v.x << 16; bits[1] = v.x & 0xFFFF0000u;
          bits[2] = v.y << 16; bits[3] = v.y & 0xFFFF0000u;
        }
        const float4 rv = *reinterpret_cast<const float4*>(rfifo + (buf * ROUNDS + r) * 32 * 16);
        float4 acc;
        acc.x = __fadd_rn(__uint_as_float(bits[0]), rv.x);
        acc.y = __fadd_rn(__uint_as_float(bits[1]), rv.y);
        acc.z = __fadd_rn(__uint_as_float(bits[2]), rv.z);
        acc.w = __fadd_rn(__uint_as_float(bits[3]), rv.w);
        *reinterpret_cast<float4*>(residual + seg_base + r * ROUND + lane * 4) = acc;
        bits[0] = __float_as_uint(acc.x); bits[1] = __float_as_uint(acc.y);
        bits[2] = __float_as_uint(acc.z); bits[3] = __float_as_uint(acc.w);
        if (src.mask != nullptr) {
          // this lane's EPL mask bits inside the round's ROUND / 32 words
          const uint32_t word = __shfl_sync(0xFFFFFFFFu, mask_words, r * (ROUND / 32) + lane * EPL / 32);
          const uint32_t m = (word >> (unsigned)((lane * EPL) & 31)) & ((1u << EPL) - 1u);
#pragma unroll
          for (int e = 0; e < EPL; ++e)
            if (m & (1u << e)) bits[e] = 0;
        }
      } else {
        // the bucket's ragged last segment: plain loads, missing elements read as 0 and are never kept
#pragma unroll
        for (int e = 0; e < EPL; ++e) {
          const unsigned long long i = seg_base + r * ROUND + lane * EPL + e;
          bits[e] = 0;
          if (i < n) {
            const float acc = __fadd_rn(__uint_as_float(src.raw1(i)), residual[i]);
            residual[i] = acc;
            bits[e] = src.pruned(i) ? 0u : __float_as_uint(acc);
          }
        }
      }
      const unsigned int f = keep_flags<EPL>(bits, t);
      if (!__any_sync(0xFFFFFFFFu, f != 0)) continue;
      kept += append_round<EPL>(f, bits, (unsigned int)(r * ROUND), seg_base + kept, seg_off, seg_val);
    }
    if (lane == 0) {
      seg_count[seg] = (unsigned short)kept;
      if (kept) atomicAdd(group_count + seg / kGroupSegs, kept);  // result unused: a fire-and-forget reduction
    }
    seg = next;
    buf ^= 1;
    mask_words = mask_words_next;
  }
  cp_async_wait<0>();
}

}  // namespace nsml
