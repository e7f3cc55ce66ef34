// Bucket -> payload without a candidate list, in one cooperative kernel.
//
// For calls that keep a large fraction of the bucket (or whose bucket is too
// small to sample) a candidate list would be about as large as the bucket, so
// the radix select (12 + 12 + 7 bits of the magnitude key; Alg. 2 Step 3 read
// as: keep the k largest |g|, ties by lower index) runs over the bucket itself.
// Block b owns the index range of its share of the 512-element segments: entry
// j of the block is element range_start + j, zeros and pruned elements included
// (they carry key 0 and take part in the selection like any other key).
//
// The range is read from memory once: phase 0 copies it into shared memory as
// far as it fits (two blocks per SM hold 2 x 23040 values, so a 25 MB float32
// bucket stays on chip entirely); what does not fit is read again from the
// bucket in every phase.  All later passes take the range four entries per
// lane at a time ("words"), each warp walking its own contiguous slice of the
// cached words and its own slice of the uncached ones, so that block order,
// warp order and lane order together are index order.
//
// Phases, separated by grid barriers (same protocol and bounds as k_finalize):
//   0  load the range, keep the shared-memory copy, histogram of digit 0   | barrier
//   1  resolve digit 0; histogram of digit 1                               | barrier
//   2  resolve digit 1; histogram of digit 2                               | barrier
//   3  resolve digit 2 -> T, r; per-warp counts of keys > T and == T       | barrier
//   4  prefix over blocks and warps; write survivors in index order
//      (float32 and fp16 values straight into the payload)
//   5  int8 only, behind one more barrier: quantise (shared with k_finalize)
#pragma once

#include "nsml_finalize.cuh"

namespace nsml {

template <int DTYPE, int THREADS, int CACHE>
__global__ void __launch_bounds__(THREADS, 1024 / THREADS)  // at most 64 registers per thread
k_finalize_dense(BucketSrc<DTYPE> src, FinalizeParams p) {
  static_assert(CACHE % 128 == 0, "a warp step (32 words) is cached as a whole or not at all");
  __shared__ FinalizeShared<THREADS, true> sh;
  extern __shared__ __align__(16) uint32_t s_cache[];
  uint4* cache4 = reinterpret_cast<uint4*>(s_cache);
  constexpr int NW = THREADS / 32;
  constexpr unsigned int CW = CACHE / 4;  // cached words
  constexpr unsigned int FULL = 0xFFFFFFFFu;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const unsigned int G = gridDim.x, blk = blockIdx.x;
  const unsigned long long range_lo = ((unsigned long long)blk * p.nseg / G) * kSegElems;  // a multiple of 512
  const unsigned long long range_hi = min(((unsigned long long)(blk + 1) * p.nseg / G) * kSegElems, p.n);
  const unsigned int E = (unsigned int)(range_hi - range_lo);  // >= 1: the grid has at most nseg blocks
  const unsigned int W = (E + 3) / 4;
  unsigned int barriers = 0;

  // This warp's slices, in words: q = 0 cached, q = 1 not cached.  Slice lengths are multiples of 32.
  const unsigned int cached_w = min(W, CW);
  unsigned int run_lo[2], run_hi[2];
  {
    const unsigned int per_a = ((cached_w + NW - 1) / NW + 31) / 32 * 32;
    const unsigned int per_b = ((W - cached_w + NW - 1) / NW + 31) / 32 * 32;
    run_lo[0] = min(cached_w, warp * per_a);
    run_hi[0] = min(cached_w, run_lo[0] + per_a);
    run_lo[1] = min(W, cached_w + warp * per_b);
    run_hi[1] = min(W, run_lo[1] + per_b);
  }

  // Entries past the end of the range inside its last word (only the bucket's ragged end has any)
  // read as zeros; this mask takes them out of every count.
  const unsigned int tail_mask = (E & 3u) ? ((1u << (E & 3u)) - 1u) : 0xFu;

  // Calls f(q, w, live, bits) for every word of the warp's slices in index order, two words per lane in
  // flight.  Within a step all 32 lanes call f (lanes past the end of the slice with live = false and
  // zero bits), so f may use warp-wide operations.
  auto for_words = [&](auto&& f) {
#pragma unroll
    for (int q = 0; q < 2; ++q) {
      for (unsigned int w0 = run_lo[q]; w0 < run_hi[q]; w0 += 64) {
        uint32_t b[2][4];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          const unsigned int w = w0 + u * 32 + lane;
          b[u][0] = b[u][1] = b[u][2] = b[u][3] = 0u;
          if (w < run_hi[q]) {
            if (q == 0) {
              const uint4 v = cache4[w];
              b[u][0] = v.x; b[u][1] = v.y; b[u][2] = v.z; b[u][3] = v.w;
            } else {
              src.load_vals4(range_lo + 4ull * w, p.n, b[u]);
            }
          }
        }
        f(q, w0 + lane, w0 + lane < run_hi[q], b[0]);
        if (w0 + 32 < run_hi[q]) f(q, w0 + 32 + lane, w0 + 32 + lane < run_hi[q], b[1]);
      }
    }
  };

  // Adds the flagged entries of a word to the shared histogram.  A warp whose 128 entries all fall
  // into one bin (a bucket of equal values) adds them with one atomic instead of 128 colliding ones.
  auto hist_add4 = [&](const unsigned int (&bin)[4], unsigned int flags) {
    const bool uniform = flags == 0xFu && bin[0] == bin[1] && bin[0] == bin[2] && bin[0] == bin[3];
    const unsigned int first = __shfl_sync(FULL, bin[0], 0);
    if (__all_sync(FULL, uniform && bin[0] == first)) {
      if (lane == 0) atomicAdd(&sh.hist[first], 128u);
      return;
    }
#pragma unroll
    for (int e = 0; e < 4; ++e)
      if (flags & (1u << e)) atomicAdd(&sh.hist[bin[e]], 1u);
  };

  // ---------------- phase 0: load the range; shared-memory copy; histogram of digit 0 ----------------
  for (int b = threadIdx.x; b < kMaxBins; b += THREADS) sh.hist[b] = 0;
  __syncthreads();
  {
    bool nonfinite = false;
    unsigned int zeros = 0;  // zero keys (pruned, embedding rows never touched) would all hit bin 0
    for (unsigned int base = 0; base < W; base += THREADS * 4) {  // four 16-byte loads in flight per thread
      uint32_t b[4][4];
      int cnt[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const unsigned int w = base + u * THREADS + threadIdx.x;
        b[u][0] = b[u][1] = b[u][2] = b[u][3] = 0u;
        cnt[u] = (w < W) ? src.load_vals4(range_lo + 4ull * w, p.n, b[u]) : 0;
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const unsigned int w = base + u * THREADS + threadIdx.x;
        if (cnt[u] != 0 && w < CW) cache4[w] = make_uint4(b[u][0], b[u][1], b[u][2], b[u][3]);
        unsigned int bin[4], flags = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const uint32_t key = b[u][e] & 0x7FFFFFFFu;
          bin[e] = key >> digit_shift(0);
          nonfinite |= key >= kInfKey;  // missing entries read as 0
          if (e < cnt[u]) {
            if (key == 0) ++zeros; else flags |= 1u << e;
          }
        }
        hist_add4(bin, flags);  // every thread of the block gets here the same number of times
      }
    }
    const unsigned long long block_zeros = block_sum(zeros, sh);
    if (threadIdx.x == 0 && block_zeros != 0) atomicAdd(&sh.hist[0], (unsigned int)block_zeros);
    if (nonfinite) set_status(&p.ctl->status, NSML_ERR_NONFINITE);
  }
  flush_hist<kMaxBins>(sh, p.hist);
  if (!grid_barrier(p.ctl, ++barriers * G, sh)) return;

  // ---------------- phase 1: resolve digit 0, histogram of digit 1 ----------------
  // Digit 0 splits the entries into those above the threshold's bin (survivors whatever T turns out
  // to be: counted here, per slice), those below it (dropped) and the undecided ones inside it.  Only
  // the undecided matter to phases 2 and 3, so each warp lists their positions (16 bits each) while it
  // is here; a warp whose list overflows, or whose positions need more than 16 bits, walks its slices
  // again instead.
  resolve_digit<kMaxBins>(p.hist, (unsigned int)p.k, sh);
  const unsigned int d0 = sh.out[0];
  unsigned int rem = sh.out[1];
  for (int b = threadIdx.x; b < kMaxBins; b += THREADS) sh.hist[b] = 0;
  __syncthreads();
  unsigned int above[2] = {0, 0};           // this lane's keys above bin d0, per slice
  unsigned int und_len = 0, und_len0 = 0;   // listed so far (warp-uniform); of those, from slice 0
  bool und_ok = E <= 65536u;                // warp-uniform
  unsigned short* und = sh.g.und[warp];
  const unsigned int lt = (1u << lane) - 1u;
  {
    unsigned int zeros = 0;
    for_words([&](int q, unsigned int w, bool live, const uint32_t (&bits)[4]) {
      unsigned int bin[4], flags = 0, zflags = 0;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const uint32_t key = bits[e] & 0x7FFFFFFFu;
        const unsigned int d = key >> 19;
        bin[e] = (key >> 7) & 0xFFFu;
        above[q] += d > d0;  // zero bits (lanes past the end, the ragged tail) are never above
        flags |= (unsigned int)(d == d0) << e;
        zflags |= (unsigned int)(key == 0) << e;
      }
      if (!live) flags = 0;
      if (w == W - 1) flags &= tail_mask;
      const unsigned int any = __ballot_sync(FULL, flags != 0);
      if (any == 0) return;  // warp-uniform
      {
        unsigned int before, total;
        if (__ballot_sync(FULL, (flags & (flags - 1)) != 0) == 0) {  // no lane has two
          before = __popc(any & lt);
          total = __popc(any);
        } else {
          const unsigned int mine = __popc(flags);
          unsigned int incl = mine;
#pragma unroll
          for (int o = 1; o < 32; o <<= 1) {
            const unsigned int up = __shfl_up_sync(FULL, incl, o);
            if (lane >= o) incl += up;
          }
          before = incl - mine;
          total = __shfl_sync(FULL, incl, 31);
        }
        if (und_ok && und_len + total <= (unsigned int)kUndCap) {
          unsigned int pos = und_len + before;
#pragma unroll
          for (int e = 0; e < 4; ++e)
            if (flags & (1u << e)) und[pos++] = (unsigned short)(4u * w + e);
        } else {
          und_ok = false;
        }
        und_len += total;
      }
      zeros += __popc(flags & zflags);  // zero keys are undecided only when d0 == 0; they would all hit bin 0
      hist_add4(bin, flags & ~zflags);
      if (q == 0) und_len0 = und_len;
    });
    const unsigned long long block_zeros = block_sum(zeros, sh);
    if (threadIdx.x == 0 && block_zeros != 0) atomicAdd(&sh.hist[0], (unsigned int)block_zeros);
  }
  flush_hist<kMaxBins>(sh, p.hist + 1 * kMaxBins);
  if (!grid_barrier(p.ctl, ++barriers * G, sh)) return;

  // Calls f(q, key) for this lane's share of the warp's listed undecided entries.
  auto for_listed = [&](auto&& f) {
    for (unsigned int i = lane; i < und_len; i += 32) {
      const unsigned int j = und[i];
      const uint32_t bits = j < (unsigned int)CACHE ? s_cache[j] : src.load1(range_lo + j);
      f(i < und_len0 ? 0 : 1, bits & 0x7FFFFFFFu);
    }
  };

  // ---------------- phase 2: resolve digit 1, histogram of digit 2 ----------------
  resolve_digit<kMaxBins>(p.hist + 1 * kMaxBins, rem, sh);
  const unsigned int prefix24 = (d0 << 12) | sh.out[0];
  rem = sh.out[1];
  __syncthreads();
  for (int b = threadIdx.x; b < 128; b += THREADS) sh.hist[b] = 0;
  __syncthreads();
  {
    unsigned int zeros = 0;
    if (und_ok) {
      for_listed([&](int, uint32_t key) {
        if ((key >> 7) != prefix24) return;
        if (key == 0) ++zeros; else atomicAdd(&sh.hist[key & 0x7Fu], 1u);
      });
    } else {
      for_words([&](int, unsigned int w, bool live, const uint32_t (&bits)[4]) {
        unsigned int bin[4], flags = 0, zflags = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const uint32_t key = bits[e] & 0x7FFFFFFFu;
          bin[e] = key & 0x7Fu;
          flags |= (unsigned int)((key >> 7) == prefix24) << e;
          zflags |= (unsigned int)(key == 0) << e;
        }
        if (!live) flags = 0;
        if (w == W - 1) flags &= tail_mask;
        zeros += __popc(flags & zflags);
        hist_add4(bin, flags & ~zflags);
      });
    }
    const unsigned long long block_zeros = block_sum(zeros, sh);
    if (threadIdx.x == 0 && block_zeros != 0) atomicAdd(&sh.hist[0], (unsigned int)block_zeros);
  }
  flush_hist<128>(sh, p.hist + 2 * kMaxBins);
  if (!grid_barrier(p.ctl, ++barriers * G, sh)) return;

  // ---------------- phase 3: T and r; this warp's keys > T and == T, per slice ----------------
  resolve_digit<128>(p.hist + 2 * kMaxBins, rem, sh);
  const uint32_t T = (prefix24 << 7) | sh.out[0];
  const unsigned int r = sh.out[1];  // ties (key == T) to keep, lowest index first
  unsigned int slice_a[2] = {0, 0}, slice_c[2] = {0, 0};  // this lane's counts, then (after the reduction) the warp's
  if (und_ok) {
    slice_a[0] = above[0];
    slice_a[1] = above[1];
    for_listed([&](int q, uint32_t key) {
      slice_a[q] += key > T;
      slice_c[q] += key == T;
    });
  } else {
    for_words([&](int q, unsigned int w, bool live, const uint32_t (&bits)[4]) {
      unsigned int fa = 0, fc = 0;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const uint32_t key = bits[e] & 0x7FFFFFFFu;
        fa |= (unsigned int)(key > T) << e;
        fc |= (unsigned int)(key == T) << e;
      }
      if (!live) fc = 0;  // zero bits are never above T, but equal it when T = 0
      if (w == W - 1) fc &= tail_mask;
      slice_a[q] += __popc(fa);
      slice_c[q] += __popc(fc);
    });
  }
#pragma unroll
  for (int q = 0; q < 2; ++q) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      slice_a[q] += __shfl_xor_sync(FULL, slice_a[q], o);
      slice_c[q] += __shfl_xor_sync(FULL, slice_c[q], o);
    }
    if (lane == 0) sh.run[q * NW + warp] = ((unsigned long long)slice_a[q] << 32) | slice_c[q];
  }
  __syncthreads();
  unsigned long long block_a = 0, block_c = 0;
  for (int w = 0; w < 2 * NW; ++w) {
    block_a += sh.run[w] >> 32;
    block_c += sh.run[w] & 0xFFFFFFFFull;
  }
  unsigned long long* ac_counts = p.block_counts + 1 * kMaxFinalizeBlocks;
  if (threadIdx.x == 0) ac_counts[blk] = (block_a << 32) | block_c;
  if (!grid_barrier(p.ctl, ++barriers * G, sh)) return;

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
  if (a_all + min(c_all, (unsigned long long)r) != p.k) {
    if (threadIdx.x == 0) set_status(&p.ctl->status, NSML_ERR_INTERNAL);
    return;
  }
  uint32_t* out_idx = reinterpret_cast<uint32_t*>(p.payload + p.P.idx_off);
  static_assert(kMaxBins * 4 >= NW * 128 * 8, "the staging areas of all warps fit the histogram");
  uint32_t* stage_idx = sh.hist + warp * 256;  // 128 indices, then 128 values, per warp
  uint32_t* stage_val = stage_idx + 128;
#pragma unroll
  for (int q = 0; q < 2; ++q) {
    // survivors before this slice: every warp's cached slice comes before any uncached one
    unsigned long long a64 = a_before, c64 = c_before;
    for (int w = 0; w < q * NW + warp; ++w) {
      a64 += sh.run[w] >> 32;
      c64 += sh.run[w] & 0xFFFFFFFFull;
    }
    unsigned int a_here = (unsigned int)a64, c_here = (unsigned int)c64;  // both < 2^31
    for (unsigned int w0 = run_lo[q]; w0 < run_hi[q]; w0 += 32) {
      const unsigned int w = w0 + lane;
      uint32_t bits[4] = {0u, 0u, 0u, 0u};
      if (w < run_hi[q]) {
        if (q == 0) {
          const uint4 v = cache4[w];
          bits[0] = v.x; bits[1] = v.y; bits[2] = v.z; bits[3] = v.w;
        } else {
          src.load_vals4(range_lo + 4ull * w, p.n, bits);
        }
      }
      unsigned int fa = 0, fc = 0;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const uint32_t key = bits[e] & 0x7FFFFFFFu;
        fa |= (unsigned int)(key > T) << e;
        fc |= (unsigned int)(key == T) << e;
      }
      if (w >= run_hi[q]) fc = 0;  // zero bits are never above T, but equal it when T = 0
      if (w == W - 1) fc &= tail_mask;
      // exclusive prefix over the lanes of (keys > T, keys == T), packed 16 + 16 bits (at most 128 each)
      const unsigned int mine = __popc(fa) | (__popc(fc) << 16);
      unsigned int incl = mine;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const unsigned int up = __shfl_up_sync(FULL, incl, o);
        if (lane >= o) incl += up;
      }
      const unsigned int total = __shfl_sync(FULL, incl, 31);
      const unsigned int a_lane = (incl - mine) & 0xFFFFu, c_lane = (incl - mine) >> 16;  // of this step, in lower lanes
      // Survivors of this step go to consecutive payload positions.  They are first put in order into the
      // warp's staging area (the histogram's shared memory, free in this phase), then written 32 at a time.
      const unsigned int c_room = r > c_here ? r - c_here : 0u;           // ties still to keep from here on
      const unsigned int ta = total & 0xFFFFu, tc = min(total >> 16, c_room);
      const unsigned int step_base = a_here + min(c_here, r);              // payload position of the step's first survivor
      if (ta + tc != 0) {  // warp-uniform
        if (fa | fc) {
          unsigned int a_rank = a_lane, c_rank = c_lane;  // within the step
          const uint32_t first_index = (uint32_t)(range_lo + 4ull * w);
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const bool is_a = fa & (1u << e), is_c = fc & (1u << e);
            if (is_a || (is_c && c_rank < c_room)) {
              const unsigned int slot = a_rank + min(c_rank, c_room);
              stage_idx[slot] = first_index + e;
              stage_val[slot] = bits[e];
            }
            a_rank += is_a;
            c_rank += is_c;
          }
        }
        __syncwarp();
        for (unsigned int i = lane; i < ta + tc; i += 32) {
          out_idx[step_base + i] = stage_idx[i];
          put_value(p, step_base + i, stage_val[i]);
        }
        __syncwarp();  // the staging area is read before the next step overwrites it
      }
      a_here += total & 0xFFFFu;
      c_here += total >> 16;
    }
  }
  // ---------------- phase 5: the header; int8: quantise ----------------
  if (blk == 0 && threadIdx.x == 0) write_header(p);
  if (p.bits != NSML_BITS_INT8) return;  // float32 and fp16 values are in the payload already
  if (!grid_barrier(p.ctl, ++barriers * G, sh)) return;
  quantize_all(p, sh);
}

}  // namespace nsml
