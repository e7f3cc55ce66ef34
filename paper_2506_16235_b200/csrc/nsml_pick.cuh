// Marked candidates -> payload, in three plain kernels (many small blocks, one
// block, many small blocks): no cooperative launch, no waiting between blocks.
//
// The bucket pass (nsml_mark.cuh) leaves a bitmap of the candidates (every key
// >= lo), their histogram over kFineBins key bins, and - resolved by its last
// block - the fine bin Tbin that holds the k-th largest key with the rank `rem`
// of that key inside the bin.  The kernels here find the exact threshold key T
// and the tie budget (Alg. 2 Step 3 read as: keep the k largest |g|, ties by
// lower index), write the k survivors in index order and quantise them (Alg. 2
// Step 1 "quantize" for fp16; int8 per block of 1024 survivors).
//
// Block b of k_pick_a and k_pick_b owns the kPickElems elements from
// b * kPickElems on, so block order is index order, nothing has to be balanced
// or agreed on, and the hardware schedules the blocks as SMs become free.
//
// A thread of these two kernels owns one bitmap round (four words, 128
// elements) of its block's range; a block-wide scan of the rounds' popcounts
// gives every thread the position of its candidates among the block's.  Every
// access to global memory costs about a microsecond of latency however little
// it moves, so each kernel issues whatever it needs in as few rounds as it can
// (control words, per-block counts and bitmap together; candidates eight at a
// time) and the grids are small enough to be resident at once.
//
// k_pick_a, per block: reads the marked elements again from the bucket
// (scattered loads, eight in flight per thread), keeps the values, in index order, in its stretch of a stash in global memory,
// and sorts each candidate into "above the threshold's bin" (a survivor
// whatever T turns out to be), "in the bin" or "below" (dropped).  If a bin holds a single
// key value (bfloat16 keys, or bins one key wide) T is the bin's key and only
// ties remain; otherwise the block appends its in-bin candidates (value, index)
// to a short global list.  It publishes its counts.
//
// k_pick_settle, one block: reads the whole list of in-bin candidates (at most
// kUndCap, typically a few hundred), finds T as the list's rem-th largest key
// and the index up to which ties at T survive, and writes for every block of
// the other two kernels the number of survivors before it.
//
// k_pick_b, per block: reads its candidates' values back from the stash, counts
// its survivors per word, scans the counts and writes the survivors' indices
// and values at their final payload positions (fp16 and float32 values
// directly; int8 values go through raw_val, and whichever block delivers the
// last survivor of a block of 1024 payload entries quantises that block - no
// waiting, no further kernel).
//
// Whatever this scheme cannot handle - fewer candidates than k (too few
// non-zero keys, or a misleading sample), more in-bin candidates or ties than
// can be listed - raises ctl->fallback; the kernels then leave at once and the
// select over the bucket itself (nsml_dense.cuh), which is enqueued behind them
// in any case and otherwise leaves at once itself, produces the payload: the
// result is exact in every case.
//
// Every global index these kernels compute is checked against its array's
// bound; a violation (which would be a bug) is recorded as NSML_ERR_INTERNAL
// and the access is skipped.
#pragma once

#include "nsml_finalize.cuh"

namespace nsml {

constexpr int kPickThreads = kPickElems / kRoundElems;  // 256: one bitmap round (128 elements) per thread
constexpr int kPickTieCap = 1024;     // ties at the threshold whose rank by index is worked out from the list
constexpr int kPickRankCap = 768;     // listed candidates up to which the threshold is found by counting ranks
constexpr int kPickQCap = 40;         // blocks of 1024 payload entries a block can complete (kPickElems / 1024 + 2 at most)
constexpr int kPickFlight = 8;        // candidates a thread fetches at a time
static_assert(kPickThreads == 256, "the quantisation takes 256 threads per block of 1024 entries");
static_assert(kPickElems <= 32768 && kPickElems / NSML_QBLOCK + 2 <= kPickQCap, "a block's survivors span at most kPickQCap payload blocks");

// rows of FinalizeParams::per_block
enum { PB_CANDS = 0, PB_ABOVE, PB_INBIN, PB_LISTED, PB_BEFORE, PB_INBIN_BEFORE };

__device__ __forceinline__ unsigned int fine_bin(uint32_t key, unsigned int lo, unsigned int shift) {
  return min((key - lo) >> shift, (unsigned int)(kFineBins - 1));
}

// Exclusive prefix over the block (kPickThreads threads) in thread order; `total` = sum over the block.
// s_warp: one word per warp.
__device__ __forceinline__ unsigned int pick_scan(unsigned int v, unsigned int& total, unsigned int* s_warp) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  unsigned int incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned int up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
    if (lane >= o) incl += up;
  }
  __syncthreads();  // s_warp may still be read from an earlier call
  if (lane == 31) s_warp[warp] = incl;
  __syncthreads();
  unsigned int before = 0, all = 0;
#pragma unroll
  for (int w = 0; w < kPickThreads / 32; ++w) {
    const unsigned int c = s_warp[w];
    if (w < warp) before += c;
    all += c;
  }
  total = all;
  return before + incl - v;
}

// This thread's bitmap round as two 64-bit masks: bit e of half h = element round_base + 64 h + e of the
// bucket is a candidate.  (No other memory access of the kernel depends on anything: issue it first.)
struct PickRound {
  unsigned long long half[2];
  unsigned long long base;  // index of the round's first element
  __device__ __forceinline__ unsigned int count() const { return __popcll(half[0]) + __popcll(half[1]); }
};
__device__ __forceinline__ PickRound pick_round(const FinalizeParams& p) {
  const unsigned long long round_id = (unsigned long long)blockIdx.x * kPickThreads + threadIdx.x;
  const unsigned long long rounds_all = (p.n + kRoundElems - 1) / kRoundElems;
  uint4 m = make_uint4(0u, 0u, 0u, 0u);
  if (round_id < rounds_all) m = __ldcg(reinterpret_cast<const uint4*>(p.bitmap) + round_id);
  PickRound r;
  r.half[0] = ((unsigned long long)m.y << 32) | m.x;
  r.half[1] = ((unsigned long long)m.w << 32) | m.z;
  r.base = round_id * kRoundElems;
  return r;
}

// Calls f(value, index) for the round's candidates in index order; their values are fetched kPickFlight at a
// time with load(position among the round's candidates, index).
template <class L, class F>
__device__ __forceinline__ void for_round_candidates(PickRound r, L&& load, F&& f) {
  unsigned int done = 0;
  while ((r.half[0] | r.half[1]) != 0) {
    uint32_t idx[kPickFlight], v[kPickFlight];
    int cnt = 0;
#pragma unroll
    for (int u = 0; u < kPickFlight; ++u) {
      idx[u] = 0;
      if (r.half[0] != 0) {
        idx[u] = (uint32_t)r.base + (__ffsll((long long)r.half[0]) - 1);
        r.half[0] &= r.half[0] - 1;
        cnt = u + 1;
      } else if (r.half[1] != 0) {
        idx[u] = (uint32_t)r.base + 64 + (__ffsll((long long)r.half[1]) - 1);
        r.half[1] &= r.half[1] - 1;
        cnt = u + 1;
      }
    }
#pragma unroll
    for (int u = 0; u < kPickFlight; ++u) v[u] = u < cnt ? load(done + u, idx[u]) : 0u;
#pragma unroll
    for (int u = 0; u < kPickFlight; ++u)
      if (u < cnt) f(v[u], idx[u]);
    done += cnt;
  }
}

template <int DTYPE>
__global__ void __launch_bounds__(kPickThreads)
k_pick_a(BucketSrc<DTYPE> src, FinalizeParams p) {
  __shared__ unsigned int s_warp[kPickThreads / 32];
  __shared__ unsigned long long s_red[kPickThreads / 32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const unsigned int blk = blockIdx.x, B = p.pick_blocks;
  Ctl* ctl = p.ctl;
  const PickRound round = pick_round(p);
  const unsigned int fallback = __ldcg(&ctl->fallback);
  const unsigned int lo = max(__ldcg(&ctl->lo), 1u), shift = __ldcg(&ctl->shift);
  const unsigned int Tbin = __ldcg(&ctl->Tbin);
  const bool by_bin = __ldcg(&ctl->by_bin) != 0;
  if (fallback != 0) return;  // the bucket pass found fewer candidates than k
  uint32_t* my_val = p.stash_val + (size_t)blk * kStashPerBlock;

  unsigned int E;
  const unsigned int first = pick_scan(round.count(), E, s_warp);  // position of this round's first candidate among the block's
  unsigned int at = first, above = 0, inbin = 0;
  bool nonfinite = false, bad = false;
  for_round_candidates(
      round,
      [&](unsigned int, uint32_t idx) { return idx < p.n ? src.raw1(idx) : 0u; },  // a candidate is never a pruned element
      [&](uint32_t v, uint32_t idx) {
        // the value goes to the stash, the key is compared with the threshold's bin
        if (at < (unsigned int)kStashPerBlock) my_val[at] = v; else bad = true;
        ++at;
        const uint32_t key = v & 0x7FFFFFFFu;
        nonfinite |= key >= kInfKey;
        if (key < lo) return;  // cannot happen: the bucket pass marked it
        const unsigned int bin = fine_bin(key, lo, shift);
        above += bin > Tbin;
        if (bin == Tbin) {
          ++inbin;
          if (!by_bin) {  // rare: a few hundred entries in the whole bucket
            const unsigned int slot = atomicAdd(&ctl->und_count, 1u);
            if (slot < kUndCap) p.und[slot] = make_uint2(v, idx);
          }
        }
      });
  if (nonfinite) set_status(&ctl->status, NSML_ERR_NONFINITE);
  if (bad) set_status(&ctl->status, NSML_ERR_INTERNAL);
  unsigned long long both = ((unsigned long long)above << 32) | inbin;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) both += __shfl_xor_sync(0xFFFFFFFFu, both, o);
  if (lane == 0) s_red[warp] = both;
  __syncthreads();
  if (threadIdx.x == 0 && blk < B) {
    both = 0;
    for (int w = 0; w < kPickThreads / 32; ++w) both += s_red[w];
    p.per_block[PB_CANDS * B + blk] = E;
    p.per_block[PB_ABOVE * B + blk] = (unsigned int)(both >> 32);
    p.per_block[PB_INBIN * B + blk] = (unsigned int)(both & 0xFFFFFFFFull);
  }
}

// One block: the exact threshold, and every block's payload position.
__global__ void __launch_bounds__(kPickThreads)
k_pick_settle(FinalizeParams p) {
  constexpr int THREADS = kPickThreads;
  constexpr int NW = THREADS / 32;
  constexpr unsigned int FULL = 0xFFFFFFFFu;
  __shared__ FinalizeShared<THREADS> sh;
  __shared__ uint2 s_u[kUndCap];  // the listed candidates
  __shared__ unsigned int s_T, s_limit;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const unsigned int B = p.pick_blocks;
  Ctl* ctl = p.ctl;
  // everything this block reads was written by the kernel before it: one round of loads
  const unsigned int fallback = __ldcg(&ctl->fallback), rem = __ldcg(&ctl->rem);
  const bool by_bin = __ldcg(&ctl->by_bin) != 0;
  const unsigned int und_all = __ldcg(&ctl->und_count);
  constexpr int kHeld = 8;  // blocks per thread whose counts are held in registers
  const unsigned int per_thread = (B + THREADS - 1) / THREADS;
  const unsigned int b_begin = min(B, threadIdx.x * per_thread), b_end = min(B, b_begin + per_thread);
  unsigned int held_above[kHeld], held_inbin[kHeld];
#pragma unroll
  for (int i = 0; i < kHeld; ++i) {
    const unsigned int b = b_begin + i;
    held_above[i] = b < b_end ? __ldcg(p.per_block + (size_t)PB_ABOVE * B + b) : 0u;
    held_inbin[i] = b < b_end ? __ldcg(p.per_block + (size_t)PB_INBIN * B + b) : 0u;
  }
  for (unsigned int i = threadIdx.x; i < min(und_all, kUndCap); i += THREADS) s_u[i] = __ldcg(p.und + i);
  if (fallback != 0) return;
  uint32_t T = 0, limit = 0;
  unsigned int ties_kept = 0;
  if (!by_bin) {
    const unsigned int und_count = und_all;
    if (und_count > kUndCap) {
      if (threadIdx.x == 0) ctl->fallback = 1u;
      return;
    }
    if (und_count < rem || rem == 0) {  // cannot happen: the bin holds at least rem keys
      if (threadIdx.x == 0) set_status(&ctl->status, NSML_ERR_INTERNAL);
      return;
    }
    // T is the rem-th largest key of the listed candidates; under (key descending, index ascending) its
    // entry has rank rem - 1.
    __syncthreads();  // the list is in shared memory
    if (und_count <= (unsigned int)kPickRankCap) {
      // short list: every entry's rank by counting, a warp per entry, the lanes share the comparisons
      for (unsigned int i = warp; i < und_count; i += NW) {
        const uint2 me = s_u[i];
        const uint32_t key = me.x & 0x7FFFFFFFu;
        unsigned int before = 0;
        for (unsigned int q = lane; q < und_count; q += 32) {
          const uint2 e = s_u[q];
          const uint32_t kq = e.x & 0x7FFFFFFFu;
          before += kq > key || (kq == key && e.y < me.y);
        }
        before = __reduce_add_sync(FULL, before);
        if (lane == 0 && before == rem - 1) {  // ranks are distinct: exactly one entry
          s_T = key;
          s_limit = me.y;
        }
      }
      __syncthreads();
      T = s_T;
      limit = s_limit;
    } else {
      // long list: radix select, 12 + 12 + 7 bits, then the rank by index among the ties at T
      unsigned int prefix = 0, left = rem;
#pragma unroll
      for (int level = 0; level < 3; ++level) {
        const int nb = 1 << digit_bits(level);
        __syncthreads();  // the previous level's bins have been read
        for (int b = threadIdx.x; b < nb; b += THREADS) sh.hist[b] = 0;
        __syncthreads();
        for (unsigned int i = threadIdx.x; i < und_count; i += THREADS) {
          const uint32_t key = s_u[i].x & 0x7FFFFFFFu;
          const bool in = level == 0 || (level == 1 ? (key >> 19) == prefix : (key >> 7) == prefix);
          if (in) atomicAdd(&sh.hist[(key >> digit_shift(level)) & (nb - 1)], 1u);
        }
        __syncthreads();
        constexpr int PER = kMaxBins / THREADS;
        unsigned int own[PER];
#pragma unroll
        for (int b = 0; b < PER; ++b) {
          const int bin = threadIdx.x * PER + b;
          own[b] = bin < nb ? sh.hist[bin] : 0u;
        }
        find_digit_from_top<PER, THREADS>(own, left, sh.tot, sh.out);
        prefix = (prefix << digit_bits(level)) | sh.out[0];
        left = sh.out[1];
      }
      T = prefix;
      const unsigned int keep = left;                // ties at T that survive, lowest index first
      const unsigned int ties = sh.hist[T & 0x7Fu];  // keys equal to T in the list
      if (keep >= ties) {
        limit = 0xFFFFFFFFu;  // every tie survives
      } else if (ties > (unsigned int)kPickTieCap) {
        if (threadIdx.x == 0) ctl->fallback = 1u;
        return;
      } else {
        // the keep-th smallest index among the ties: the one with keep - 1 tied indices below it
        for (unsigned int i = threadIdx.x; i < und_count; i += THREADS) {
          const uint2 me = s_u[i];
          if ((me.x & 0x7FFFFFFFu) != T) continue;
          unsigned int below = 0;
          for (unsigned int q = 0; q < und_count; ++q) {
            const uint2 e = s_u[q];
            below += (e.x & 0x7FFFFFFFu) == T && e.y < me.y;
          }
          if (below == keep - 1) s_limit = me.y;  // indices are distinct: exactly one thread
        }
        __syncthreads();
        limit = s_limit;
      }
    }
    // listed survivors per block
    unsigned int* listed = p.per_block + (size_t)PB_LISTED * B;
    for (unsigned int b = threadIdx.x; b < B; b += THREADS) listed[b] = 0;
    __syncthreads();
    for (unsigned int i = threadIdx.x; i < und_count; i += THREADS) {
      const uint2 e = s_u[i];
      const uint32_t key = e.x & 0x7FFFFFFFu;
      const unsigned int owner = e.y / (unsigned int)kPickElems;
      if ((key > T || (key == T && e.y <= limit)) && owner < B) atomicAdd(listed + owner, 1u);
    }
    __syncthreads();
  }
  // Exclusive prefix over the blocks of (sure survivors [+ listed survivors], in-bin entries): every thread
  // takes a contiguous range of blocks, sums it (independent loads), the sums are scanned over the block,
  // and a second walk writes the prefixes.
  auto value_of = [&](unsigned int b) {  // blocks beyond the held ones
    unsigned int s = __ldcg(p.per_block + (size_t)PB_ABOVE * B + b);
    if (!by_bin) s += __ldcg(p.per_block + (size_t)PB_LISTED * B + b);
    return ((unsigned long long)s << 32) | __ldcg(p.per_block + (size_t)PB_INBIN * B + b);
  };
  unsigned long long held[kHeld];
#pragma unroll
  for (int i = 0; i < kHeld; ++i) {
    const unsigned int b = b_begin + i;
    unsigned int s = held_above[i];
    if (!by_bin && b < b_end) s += __ldcg(p.per_block + (size_t)PB_LISTED * B + b);  // written by this block, above
    held[i] = ((unsigned long long)s << 32) | held_inbin[i];
  }
  unsigned long long mine = 0;
#pragma unroll
  for (int i = 0; i < kHeld; ++i) mine += held[i];
  for (unsigned int b = b_begin + kHeld; b < b_end; ++b) mine += value_of(b);
  unsigned long long incl = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned long long up = __shfl_up_sync(FULL, incl, o);
    if (lane >= o) incl += up;
  }
  __syncthreads();
  if (lane == 31) sh.red[warp] = incl;
  __syncthreads();
  unsigned long long run = incl - mine, carry = 0;
#pragma unroll
  for (int w = 0; w < NW; ++w) {
    const unsigned long long c = sh.red[w];
    if (w < warp) run += c;
    carry += c;
  }
#pragma unroll
  for (int i = 0; i < kHeld; ++i) {
    const unsigned int b = b_begin + i;
    if (b < b_end) {
      p.per_block[PB_BEFORE * B + b] = (unsigned int)(run >> 32);
      p.per_block[PB_INBIN_BEFORE * B + b] = (unsigned int)(run & 0xFFFFFFFFull);
    }
    run += held[i];
  }
  for (unsigned int b = b_begin + kHeld; b < b_end; ++b) {
    p.per_block[PB_BEFORE * B + b] = (unsigned int)(run >> 32);
    p.per_block[PB_INBIN_BEFORE * B + b] = (unsigned int)(run & 0xFFFFFFFFull);
    run += value_of(b);
  }
  const unsigned long long sure = carry >> 32, in_all = carry & 0xFFFFFFFFull;
  if (by_bin) {
    // every in-bin key equals T: the first k - sure of them in index order survive
    if (sure > p.k || in_all < p.k - sure) {  // cannot happen: the histogram put the k-th largest key into this bin
      if (threadIdx.x == 0) set_status(&ctl->status, NSML_ERR_INTERNAL);
      return;
    }
    ties_kept = (unsigned int)(p.k - sure);
  } else if (sure != p.k) {  // cannot happen
    if (threadIdx.x == 0) set_status(&ctl->status, NSML_ERR_INTERNAL);
    return;
  }
  if (threadIdx.x == 0) {
    ctl->T = T;
    ctl->limit = limit;
    ctl->ties_kept = ties_kept;
  }
}

__global__ void __launch_bounds__(kPickThreads)
k_pick_b(FinalizeParams p) {
  constexpr int THREADS = kPickThreads;
  constexpr int NW = THREADS / 32;
  struct Scratch {
    float qmax[NW];  // the quantisation's scratch
  };
  __shared__ Scratch sh;
  __shared__ unsigned int s_warp[NW];
  __shared__ unsigned int s_q[kPickQCap];
  __shared__ unsigned int s_nq;
  const unsigned int blk = blockIdx.x, B = p.pick_blocks;
  const Ctl* ctl = p.ctl;
  // everything this block reads first was written by the kernels before it: one round of loads
  const PickRound round = pick_round(p);
  const unsigned int fallback = __ldcg(&ctl->fallback);
  const int status = __ldcg(&ctl->status);
  const unsigned int lo = max(__ldcg(&ctl->lo), 1u), shift = __ldcg(&ctl->shift), Tbin = __ldcg(&ctl->Tbin);
  const bool by_bin = __ldcg(&ctl->by_bin) != 0;
  const uint32_t T = __ldcg(&ctl->T), limit = __ldcg(&ctl->limit);
  const unsigned long long r = __ldcg(&ctl->ties_kept);  // by-bin case: ties (key == T) to keep, lowest index first
  const unsigned long long a_before = __ldcg(p.per_block + (size_t)PB_BEFORE * B + blk);
  const unsigned long long c_before_all = __ldcg(p.per_block + (size_t)PB_INBIN_BEFORE * B + blk);
  if (fallback != 0 || status == NSML_ERR_INTERNAL) return;
  const unsigned long long c_before = by_bin ? c_before_all : 0ull;
  if (blk == 0 && threadIdx.x == 0) write_header(p);
  const uint32_t* my_val = p.stash_val + (size_t)blk * kStashPerBlock;
  uint32_t* out_idx = reinterpret_cast<uint32_t*>(p.payload + p.P.idx_off);

  unsigned int E;
  const unsigned int first = pick_scan(round.count(), E, s_warp);  // this round's first candidate in the stash
  // a: survives whatever the ties' ranks; c: a tie at T in the by-bin case (survives while the budget lasts)
  auto classify = [&](uint32_t v, uint32_t idx, bool& a, bool& c) {
    const uint32_t key = v & 0x7FFFFFFFu;
    const bool cand = key >= lo;
    const unsigned int bin = cand ? fine_bin(key, lo, shift) : 0u;
    if (by_bin) {
      a = cand && bin > Tbin;
      c = cand && bin == Tbin;
    } else {
      a = cand && (bin > Tbin || (bin == Tbin && (key > T || (key == T && idx <= limit))));
      c = false;
    }
  };
  auto from_stash = [&](unsigned int j, uint32_t) {
    return first + j < (unsigned int)kStashPerBlock ? __ldcg(my_val + first + j) : 0u;
  };
  unsigned int my_a = 0, my_c = 0;  // at most 128 each
  for_round_candidates(round, from_stash, [&](uint32_t v, uint32_t idx) {
    bool a, c;
    classify(v, idx, a, c);
    my_a += a;
    my_c += c;
  });
  unsigned int packed_all;
  const unsigned int packed_before = pick_scan(my_a | (my_c << 16), packed_all, s_warp);  // at most kPickElems each: 16 bits do
  unsigned long long a_mine = a_before + (packed_before & 0xFFFFu), c_mine = c_before + (packed_before >> 16);
  bool bad = false;
  for_round_candidates(round, from_stash, [&](uint32_t v, uint32_t idx) {
    bool a, c;
    classify(v, idx, a, c);
    if (a || (c && c_mine < r)) {
      const unsigned long long pos = a_mine + min(c_mine, r);
      if (pos < p.k) {
        out_idx[pos] = idx;
        if (p.bits == NSML_BITS_FP32) reinterpret_cast<uint32_t*>(p.payload + p.P.val_off)[pos] = v;
        else if (p.bits == NSML_BITS_FP16) reinterpret_cast<uint16_t*>(p.payload + p.P.val_off)[pos] = encode_f16(__uint_as_float(v));
        else p.raw_val[pos] = __uint_as_float(v);
      } else {
        bad = true;
      }
    }
    a_mine += a;
    c_mine += c;
  });
  if (bad) set_status(&p.ctl->status, NSML_ERR_INTERNAL);
  // payload positions [p0, p1) of this block's survivors
  const unsigned long long p0 = a_before + min(c_before, r);
  const unsigned long long p1 = a_before + (packed_all & 0xFFFFu) + min(c_before + (packed_all >> 16), r);
  if (p.bits != NSML_BITS_INT8 || p1 <= p0 || p1 > p.k) return;  // block-uniform

  // ---------------- int8: whoever completes a block of 1024 payload entries quantises it ----------------
  __threadfence();  // this thread's raw values are visible device-wide before the block reports them
  if (threadIdx.x == 0) s_nq = 0;
  __syncthreads();
  const unsigned long long q_first = p0 / NSML_QBLOCK, q_last = (p1 - 1) / NSML_QBLOCK;
  for (unsigned long long q = q_first + threadIdx.x; q <= q_last; q += THREADS) {
    const unsigned long long q_lo = q * NSML_QBLOCK, q_hi = min(q_lo + NSML_QBLOCK, p.k);
    const unsigned int part = (unsigned int)(min(p1, q_hi) - max(p0, q_lo));
    const unsigned int seen = atomicAdd(p.qcount + q, part);
    if (seen + part == (unsigned int)(q_hi - q_lo)) {
      const unsigned int slot = atomicAdd(&s_nq, 1u);
      if (slot < (unsigned int)kPickQCap) s_q[slot] = (unsigned int)q;
    }
  }
  __syncthreads();
  __threadfence();  // the other blocks' raw values, reported before ours, are visible to the loads below
  const unsigned int nq = min(s_nq, (unsigned int)kPickQCap);
  for (unsigned int i = 0; i < nq; ++i) quantize_block(p, sh, s_q[i], true);  // 256 threads: one group
}

}  // namespace nsml
