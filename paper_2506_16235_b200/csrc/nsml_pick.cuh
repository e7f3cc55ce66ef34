// Marked candidates -> payload, in one cooperative kernel with ONE grid barrier.
//
// The bucket pass (nsml_mark.cuh) leaves a bitmap of the candidates (every key
// >= lo), their number per group of kGroupElems elements and their histogram
// over kFineBins key bins.  This kernel finds the exact threshold key T and the
// tie budget r (Alg. 2 Step 3 read as: keep the k largest |g|, ties by lower
// index), writes the k survivors in index order and quantises them (Alg. 2
// Step 1 "quantize" for fp16; int8 per block of 1024 survivors).
//
// Before the barrier, every block for itself:
//   - resolves the fine bin that holds the k-th largest key (the histogram is
//     complete: it was built by the previous kernel);
//   - scans the group counts, which gives it an equal share of the candidates
//     as a run of whole groups (block order = index order, and the work is
//     balanced however the candidates crowd into a few tensors);
//   - expands its groups' bitmap words into a list of indices in shared
//     memory and reads those elements again from the bucket (scattered loads,
//     all in flight at once), keeping the values in shared memory too (a share
//     that does not fit shared memory is kept in a spill area in global memory);
//   - sorts each candidate into "above the threshold's bin" (a survivor whatever
//     T turns out to be), "in the bin" or "below" (dropped).
//   If a bin holds a single key value (bfloat16 keys, or bins one key wide) T is
//   the bin's key and only ties remain: the block publishes its counts of keys
//   > T and == T.  Otherwise it appends its in-bin candidates (value, index) to
//   a short global list and publishes its count of keys above the bin.
// After the barrier, every block for itself:
//   - sums the other blocks' counts (survivors before its own first one);
//   - in the second case reads the whole list of in-bin candidates (at most
//     kUndCap, typically a few hundred), radix-selects T among them, finds the
//     index up to which ties at T survive, and counts the list's survivors
//     that lie before its own index range;
//   - writes its survivors' indices and values at their final payload
//     positions (fp16 and float32 values directly; int8 values go through
//     raw_val, and whichever block delivers the last survivor of a block of
//     1024 payload entries quantises that block - no waiting, no third phase).
//
// Whatever this scheme cannot handle - fewer candidates than k (too few
// non-zero keys, or a misleading sample), a table that does not fit shared
// memory, more in-bin candidates or ties than can be listed - is
// detected by every block alike, and the launch then runs the select over the
// bucket itself (nsml_dense.cuh) instead: the result is exact in every case.
#pragma once

#include "nsml_dense.cuh"
#include "nsml_finalize.cuh"

namespace nsml {

constexpr int kPickThreads = 256;
constexpr int kPickGroupCap = 1024;   // groups a block can own
constexpr int kPickTieCap = 1024;     // ties at the threshold whose rank by index is worked out from the list
constexpr int kPickRankCap = 768;     // listed candidates up to which the threshold is found by counting ranks
constexpr int kPickInbinCap = 16;     // in-bin candidates a warp remembers (more: it walks its run again)
constexpr int kPickQCap = 64;         // blocks of 1024 payload entries a block can complete
constexpr int kGroupRounds = kGroupElems / kRoundElems;  // 64
// shared memory of the list stage for a block that holds `cap` candidates: indices, values, the undecided list
constexpr size_t pick_dyn_smem(unsigned int cap) { return (size_t)cap * 8 + (size_t)kUndCap * 8; }

template <int DTYPE>
__global__ void __launch_bounds__(kPickThreads, 4)  // at most 64 registers per thread: a quarter of an SM's register file
k_pick(BucketSrc<DTYPE> src, FinalizeParams p) {
  constexpr int THREADS = kPickThreads;
  constexpr int NW = THREADS / 32;
  constexpr unsigned int FULL = 0xFFFFFFFFu;
  __shared__ FinalizeShared<THREADS> sh;
  __shared__ unsigned int s_groups[kPickGroupCap];
  __shared__ unsigned int s_q[kPickQCap];
  __shared__ unsigned int s_nq, s_limit, s_T;
  __shared__ unsigned int s_inbin[kPickThreads / 32][kPickInbinCap];  // positions of a warp's candidates in the threshold's bin
  extern __shared__ __align__(16) uint32_t s_dyn[];
  uint32_t* c_idx = s_dyn;
  uint32_t* c_val = s_dyn + p.cap;
  uint2* s_u = reinterpret_cast<uint2*>(s_dyn + 2 * (size_t)p.cap);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const unsigned int lt = (1u << lane) - 1u;
  const unsigned int G = gridDim.x, blk = blockIdx.x;
  const unsigned int lo = max(p.ctl->lo, 1u), shift = p.ctl->shift;
  bool give_up = false;  // block-uniform
  bool in_shared = true;  // the block's candidates are held in shared memory (else in the spill area)

  // ---------------- the threshold's fine bin; this block's share: a run of whole groups ----------------
  // The histogram and the group counts are both complete (the previous kernel built them): their loads are
  // issued together.  The group counts are staged in the shared memory that will hold the candidates.
  unsigned int Tbin = 0, rem = 0;  // rem: rank of the threshold inside its bin, from the top
  unsigned long long total;
  unsigned int E = 0;              // candidates this block owns
  unsigned int owned_all = 0;      // groups this block owns
  {
    constexpr int PER = kFineBins / THREADS;
    unsigned int own[PER], mine = 0;
#pragma unroll
    for (int b = 0; b < PER; ++b) own[b] = __ldcg(p.fine + (size_t)(threadIdx.x * PER + b) * kFineStride);
    uint32_t* staged = s_dyn;  // group counts, when they fit
    const bool stage = p.ngroups <= 2 * p.cap;
    if (stage)
      for (unsigned int g = threadIdx.x; g < p.ngroups; g += THREADS) staged[g] = __ldcg(p.group_count + g);
#pragma unroll
    for (int b = 0; b < PER; ++b) mine += own[b];
    total = block_sum((unsigned long long)mine, sh);  // (its barriers also complete the staging)
    if (total < p.k) {
      give_up = true;  // fewer candidates than survivors
    } else {
      find_digit_from_top<PER, THREADS>(own, (unsigned int)p.k, sh.tot, sh.out);
      Tbin = sh.out[0];
      rem = sh.out[1];
    }
    if (!give_up) {
      auto count_of = [&](unsigned int g) { return stage ? staged[g] : __ldcg(p.group_count + g); };
      // A block's work is its candidates plus the bitmap rounds of its groups, so the groups are dealt out
      // by weight: candidates + kGroupRounds for a group that has any, nothing for an empty one.
      auto weight_of = [&](unsigned int c) { return c != 0 ? c + (unsigned int)kGroupRounds : 0u; };
      const unsigned int per_thread = (p.ngroups + THREADS - 1) / THREADS;
      const unsigned int g_begin = min(p.ngroups, threadIdx.x * per_thread);
      const unsigned int g_end = min(p.ngroups, g_begin + per_thread);
      unsigned int thread_sum = 0;
      for (unsigned int g = g_begin; g < g_end; ++g) thread_sum += weight_of(count_of(g));
      unsigned int all;
      const unsigned int thread_pos = block_excl_scan(thread_sum, all, sh);  // weight before this thread's groups
      // a group belongs to the block into whose share [w_lo, w_hi) of the weight its start falls
      const unsigned long long w_lo = (unsigned long long)blk * all / G, w_hi = (unsigned long long)(blk + 1) * all / G;
      unsigned int owned = 0, owned_cands = 0, earlier_cands = 0, pos = thread_pos;
      for (unsigned int g = g_begin; g < g_end; ++g) {
        const unsigned int c = count_of(g);
        if (c != 0 && pos >= w_lo && pos < w_hi) {
          ++owned;
          owned_cands += c;
        }
        if (pos < w_lo) earlier_cands += c;
        pos += weight_of(c);
      }
      unsigned int slot = block_excl_scan(owned, owned_all, sh);
      const unsigned long long both = block_sum(((unsigned long long)earlier_cands << 32) | owned_cands, sh);
      E = (unsigned int)(both & 0xFFFFFFFFull);
      const unsigned long long cands_before = both >> 32;  // candidates of the blocks before this one
      if (E > p.cap) {
        // a share too large for shared memory lives in the spill area (its own stretch of it: blocks are in
        // index order, so the candidates before this block's say where)
        in_shared = false;
        c_idx = p.spill_idx + cands_before;
        c_val = p.spill_val + cands_before;
      }
      if (owned_all > (unsigned int)kPickGroupCap || (!in_shared && cands_before + E > p.spill_entries)) {
        give_up = true;
      } else {
        pos = thread_pos;
        for (unsigned int g = g_begin; g < g_end; ++g) {
          const unsigned int c = count_of(g);
          if (c != 0 && pos >= w_lo && pos < w_hi) s_groups[slot++] = g;
          pos += weight_of(c);
        }
      }
      __syncthreads();  // the list of groups is complete, and the staged counts have been read for the last time
    }
  }
  // a bin below the last holds exactly one key value when the sample kernel said so
  // (then the bin itself decides: above it = above T, in it = equal to T)
  const bool exact = p.ctl->exact != 0 && Tbin + 1 < (unsigned int)kFineBins;
  {
    // ---------------- bitmap -> indices, in index order ----------------
    if (!give_up) {
      const unsigned long long rounds_all = (p.n + kRoundElems - 1) / kRoundElems;
      const unsigned int nrounds = owned_all * kGroupRounds;
      const uint4* bitmap4 = reinterpret_cast<const uint4*>(p.bitmap);
      unsigned int filled = 0;
      // A thread takes `rpt` consecutive rounds per pass: one when the block's groups are few (they are then
      // crowded with candidates, and writing out a round's indices is the long part), up to RP when the
      // block owns many sparse groups (so that one pass, with its one block-wide scan, usually does).
      constexpr int RP = 8;
      const unsigned int rpt = min((unsigned int)RP, (nrounds + THREADS - 1) / THREADS);
      for (unsigned int r0 = 0; r0 < nrounds; r0 += THREADS * rpt) {
        uint4 m[RP];
        unsigned long long round_id[RP];
        unsigned int cnt = 0;
#pragma unroll
        for (int u = 0; u < RP; ++u) {
          const unsigned int r = r0 + threadIdx.x * rpt + u;
          m[u] = make_uint4(0u, 0u, 0u, 0u);
          round_id[u] = 0;
          if ((unsigned int)u < rpt && r < nrounds) {
            round_id[u] = (unsigned long long)s_groups[r / kGroupRounds] * kGroupRounds + r % kGroupRounds;
            if (round_id[u] < rounds_all) m[u] = __ldcg(bitmap4 + round_id[u]);
          }
        }
#pragma unroll
        for (int u = 0; u < RP; ++u) cnt += __popc(m[u].x) + __popc(m[u].y) + __popc(m[u].z) + __popc(m[u].w);
        unsigned int step_total;
        unsigned int at = filled + block_excl_scan(cnt, step_total, sh);
#pragma unroll
        for (int u = 0; u < RP; ++u) {
          const uint32_t first = (uint32_t)(round_id[u] * kRoundElems);
          const unsigned int words[4] = {m[u].x, m[u].y, m[u].z, m[u].w};
#pragma unroll
          for (int w = 0; w < 4; ++w) {
            unsigned int bits = words[w];
            while (bits != 0) {
              const int b = __ffs(bits) - 1;
              bits &= bits - 1;
              if (at < E) c_idx[at] = first + w * 32 + b;
              ++at;
            }
          }
        }
        filled += step_total;
      }
      if (filled != E) give_up = true;  // bitmap and counts disagree - cannot happen
    }
  }
  __syncthreads();

  // ---------------- values of the candidates; where each stands against the threshold's bin ----------------
  // Each warp owns one contiguous run of the block's candidates, so that warp order and lane order are
  // index order.  A run's counts stay in shared memory for the write phase.
  const unsigned int per_run = ((E + NW - 1) / NW + 31) / 32 * 32;
  const unsigned int run_lo = min(E, warp * per_run), run_hi = min(E, run_lo + per_run);
  unsigned int n_inbin = 0;  // this warp's candidates in the threshold's bin (listed case; warp-uniform)
  unsigned int above_run = 0;  // this warp's candidates above the bin
  if (!give_up) {
    bool nonfinite = false;
    for (unsigned int j0 = threadIdx.x; j0 < E; j0 += THREADS * 4) {  // four scattered loads in flight per thread
      uint32_t v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const unsigned int j = j0 + u * THREADS;
        v[u] = (j < E) ? src.raw1(c_idx[j]) : 0u;  // a candidate is never a pruned element
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const unsigned int j = j0 + u * THREADS;
        if (j < E) c_val[j] = v[u];
        nonfinite |= (v[u] & 0x7FFFFFFFu) >= kInfKey;
      }
    }
    if (nonfinite) set_status(&p.ctl->status, NSML_ERR_NONFINITE);
    __syncthreads();
    unsigned int wa = 0, wc = 0;
    for (unsigned int j0 = run_lo; j0 < run_hi; j0 += 32) {
      const unsigned int j = j0 + lane;
      const bool live = j < run_hi;
      const uint32_t bits = live ? c_val[j] : 0u;
      const uint32_t key = bits & 0x7FFFFFFFu;
      const unsigned int bin = (live && key >= lo) ? min((key - lo) >> shift, (unsigned int)(kFineBins - 1)) : 0u;
      const bool above = live && key >= lo && bin > Tbin;
      const bool inbin = live && key >= lo && bin == Tbin;
      wa += __popc(__ballot_sync(FULL, above));
      const unsigned int bi = __ballot_sync(FULL, inbin);
      if (exact) {
        wc += __popc(bi);  // in the bin = equal to T
      } else if (bi != 0) {
        unsigned int base = 0;
        if (lane == 0) base = atomicAdd(&p.ctl->und_count, (unsigned int)__popc(bi));
        base = __shfl_sync(FULL, base, 0);
        const unsigned int at = base + __popc(bi & lt);
        if (inbin && at < kUndCap) p.und[at] = make_uint2(bits, c_idx[j]);
        const unsigned int mine = n_inbin + __popc(bi & lt);
        if (inbin && mine < (unsigned int)kPickInbinCap) s_inbin[warp][mine] = j;
        n_inbin += __popc(bi);
      }
    }
    above_run = wa;
    if (lane == 0) sh.run[warp] = ((unsigned long long)wa << 32) | wc;
    __syncthreads();
    if (threadIdx.x == 0) {
      unsigned long long block_a = 0, block_c = 0;
      for (int w = 0; w < NW; ++w) {
        block_a += sh.run[w] >> 32;
        block_c += sh.run[w] & 0xFFFFFFFFull;
      }
      p.block_counts[blk] = (block_a << 32) | block_c;
    }
  }
  if (give_up && threadIdx.x == 0) atomicOr(&p.ctl->fallback, 1u);
  if (!grid_barrier(p.ctl, G, sh)) return;

  // =============================== after the barrier ===============================
  const unsigned int und_count = __ldcg(&p.ctl->und_count);
  bool fallback = __ldcg(&p.ctl->fallback) != 0 || und_count > kUndCap;  // the same in every block
  unsigned long long a_before = 0, c_before = 0, a_all = 0, c_all = 0;
  if (!fallback) {
    for (unsigned int b = threadIdx.x; b < G; b += THREADS) {
      const unsigned long long w = __ldcg(p.block_counts + b);
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
  }

  // ---------------- the exact threshold ----------------
  uint32_t T = 0;               // listed candidates: the threshold key
  unsigned long long r = 0;     // exact bins: ties (key == T) to keep, lowest index first
  bool limited = false;         // listed candidates: ties at T survive only up to index `limit`
  uint32_t limit = 0;
  unsigned long long u_before = 0;  // listed candidates that survive and lie before this block's index range
  if (!fallback && exact) {
    r = p.k - a_all;
    if (a_all > p.k || c_all < r) {  // cannot happen: the histogram put the k-th largest key into this bin
      if (threadIdx.x == 0) set_status(&p.ctl->status, NSML_ERR_INTERNAL);
      return;
    }
  } else if (!fallback) {
    // every block reads the whole list and selects the rem-th largest key in it: 12 + 12 + 7 bits
    for (unsigned int i = threadIdx.x; i < und_count; i += THREADS) s_u[i] = __ldcg(p.und + i);
    if (a_all + und_count < p.k || a_all >= p.k || p.k - a_all != rem) {  // cannot happen
      if (threadIdx.x == 0) set_status(&p.ctl->status, NSML_ERR_INTERNAL);
      return;
    }
    __syncthreads();  // the list is in place
    if (und_count <= (unsigned int)kPickRankCap) {
      // short list: every entry's rank under (key descending, index ascending) by counting; the entry of
      // rank rem - 1 is the last survivor: its key is T, its index the limit for ties at T
      for (unsigned int i = warp; i < und_count; i += NW) {  // a warp per entry, the lanes share the comparisons
        const uint32_t key = s_u[i].x & 0x7FFFFFFFu, idx = s_u[i].y;
        unsigned int before = 0;
        for (unsigned int q = lane; q < und_count; q += 32) {
          const uint2 e = s_u[q];
          const uint32_t kq = e.x & 0x7FFFFFFFu;
          before += kq > key || (kq == key && e.y < idx);
        }
        before = __reduce_add_sync(FULL, before);
        if (lane == 0 && before == rem - 1) {  // ranks are distinct: exactly one entry
          s_T = key;
          s_limit = idx;
        }
      }
      __syncthreads();
      T = s_T;
      limit = s_limit;
      limited = true;
    } else {
      unsigned int prefix = 0, left = rem;
#pragma unroll
      for (int level = 0; level < 3; ++level) {
        const int nb = 1 << digit_bits(level);
        __syncthreads();  // the list is in place; the previous level's bins have been read
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
      const unsigned int keep_ties = left;          // ties at T that survive, lowest index first
      const unsigned int ties = sh.hist[T & 0x7Fu];  // keys equal to T in the list
      limited = keep_ties < ties;
      if (limited && ties > (unsigned int)kPickTieCap) {
        fallback = true;  // the same decision in every block: they all hold the same list
      } else if (limited) {
        // the keep_ties-th smallest index among the ties: the one with keep_ties - 1 tied indices below it
        for (unsigned int i = threadIdx.x; i < und_count; i += THREADS) {
          if ((s_u[i].x & 0x7FFFFFFFu) != T) continue;
          const uint32_t mine = s_u[i].y;
          unsigned int below = 0;
          for (unsigned int q = 0; q < und_count; ++q) below += (s_u[q].x & 0x7FFFFFFFu) == T && s_u[q].y < mine;
          if (below == keep_ties - 1) s_limit = mine;  // indices are distinct: exactly one thread
        }
        __syncthreads();
        limit = s_limit;
      }
    }
    if (!fallback) {
      const uint32_t my_first = E != 0 ? c_idx[0] : 0xFFFFFFFFu;
      unsigned int before = 0;
      for (unsigned int i = threadIdx.x; i < und_count; i += THREADS) {
        const uint32_t key = s_u[i].x & 0x7FFFFFFFu;
        const bool survives = key > T || (key == T && (!limited || s_u[i].y <= limit));
        before += survives && s_u[i].y < my_first;
      }
      u_before = block_sum((unsigned long long)before, sh);
    }
  }

  if (fallback) {
    // select over the bucket itself; the shared memory of the list stage becomes its value cache
    dense_select<DTYPE, THREADS>(src, p, sh, s_dyn, 1u);
    return;
  }

  // ---------------- write the survivors in index order ----------------
  if (blk == 0 && threadIdx.x == 0) write_header(p);
  auto survives_listed = [&](uint32_t key, uint32_t idx) {  // a candidate in the threshold's bin, listed case
    return key > T || (key == T && (!limited || idx <= limit));
  };
  if (!exact) {
    // survivors per run, now that T is known: those above the bin plus the in-bin ones that pass
    unsigned int wa = above_run;
    if (n_inbin <= (unsigned int)kPickInbinCap) {
      bool s = false;
      if ((unsigned int)lane < n_inbin) {
        const unsigned int j = s_inbin[warp][lane];
        s = survives_listed(c_val[j] & 0x7FFFFFFFu, c_idx[j]);
      }
      wa += __popc(__ballot_sync(FULL, s));
    } else {
      wa = 0;
      for (unsigned int j0 = run_lo; j0 < run_hi; j0 += 32) {
        const unsigned int j = j0 + lane;
        bool s = false;
        if (j < run_hi) {
          const uint32_t key = c_val[j] & 0x7FFFFFFFu;
          const unsigned int bin = key >= lo ? min((key - lo) >> shift, (unsigned int)(kFineBins - 1)) : 0u;
          s = key >= lo && (bin > Tbin || (bin == Tbin && survives_listed(key, c_idx[j])));
        }
        wa += __popc(__ballot_sync(FULL, s));
      }
    }
    __syncthreads();  // sh.run of the first phase has been read by thread 0
    if (lane == 0) sh.run[warp] = (unsigned long long)wa << 32;
    __syncthreads();
  }
  unsigned long long a_here = a_before + u_before, c_here = c_before, block_a = 0, block_c = 0;
  for (int w = 0; w < NW; ++w) {
    const unsigned long long rw = sh.run[w];
    if (w < warp) {
      a_here += rw >> 32;
      c_here += rw & 0xFFFFFFFFull;
    }
    block_a += rw >> 32;
    block_c += rw & 0xFFFFFFFFull;
  }
  // payload positions [p0, p1) of this block's survivors
  const unsigned long long p0 = a_before + u_before + min(c_before, r);
  const unsigned long long p1 = a_before + u_before + block_a + min(c_before + block_c, r);
  if (blk == G - 1 && p1 != p.k) {  // cannot happen
    if (threadIdx.x == 0) set_status(&p.ctl->status, NSML_ERR_INTERNAL);
    return;
  }
  uint32_t* out_idx = reinterpret_cast<uint32_t*>(p.payload + p.P.idx_off);
  for (unsigned int j0 = run_lo; j0 < run_hi; j0 += 32) {
    const unsigned int j = j0 + lane;
    const bool live = j < run_hi;
    const uint32_t bits = live ? c_val[j] : 0u;
    const uint32_t idx = live ? c_idx[j] : 0u;
    const uint32_t key = bits & 0x7FFFFFFFu;
    const unsigned int bin = (live && key >= lo) ? min((key - lo) >> shift, (unsigned int)(kFineBins - 1)) : 0u;
    const bool cand = live && key >= lo;
    bool a, c;
    if (exact) {
      a = cand && bin > Tbin;
      c = cand && bin == Tbin;
    } else {
      a = cand && (bin > Tbin || (bin == Tbin && survives_listed(key, idx)));
      c = false;
    }
    const unsigned int ba = __ballot_sync(FULL, a), bc = __ballot_sync(FULL, c);
    const unsigned long long a_mine = a_here + __popc(ba & lt), c_mine = c_here + __popc(bc & lt);
    if (a || (c && c_mine < r)) {
      const unsigned long long pos = a_mine + min(c_mine, r);
      out_idx[pos] = idx;
      if (p.bits == NSML_BITS_FP32) reinterpret_cast<uint32_t*>(p.payload + p.P.val_off)[pos] = bits;
      else if (p.bits == NSML_BITS_FP16) reinterpret_cast<uint16_t*>(p.payload + p.P.val_off)[pos] = encode_f16(__uint_as_float(bits));
      else p.raw_val[pos] = __uint_as_float(bits);
    }
    a_here += __popc(ba);
    c_here += __popc(bc);
  }
  if (p.bits != NSML_BITS_INT8 || p1 == p0) return;  // block-uniform

  // ---------------- int8: whoever completes a block of 1024 payload entries quantises it ----------------
  __threadfence();  // this thread's raw values are visible device-wide before the block reports them
  if (threadIdx.x == 0) s_nq = 0;
  __syncthreads();
  const unsigned long long q_first = p0 / NSML_QBLOCK, q_last = (p1 - 1) / NSML_QBLOCK;
  for (unsigned long long q = q_first + threadIdx.x; q <= q_last; q += THREADS) {
    const unsigned long long q_lo = q * NSML_QBLOCK, q_hi = min(q_lo + NSML_QBLOCK, p.k);
    const unsigned int part = (unsigned int)(min(p1, q_hi) - max(p0, q_lo));
    const unsigned int seen = atomicAdd(p.qcount + q, part);
    if (seen + part == (unsigned int)(q_hi - q_lo)) s_q[atomicAdd(&s_nq, 1u)] = (unsigned int)q;  // at most kPickQCap: cap / 1024 + 2
  }
  __syncthreads();
  __threadfence();  // the other blocks' raw values, reported before ours, are visible to the loads below
  const unsigned int nq = s_nq;
  constexpr int kQGroups = THREADS / 256;
  for (unsigned int i0 = 0; i0 < nq; i0 += kQGroups) {
    const unsigned int i = i0 + (threadIdx.x >> 8);
    quantize_block(p, sh, i < nq ? s_q[i] : 0ull, i < nq);
  }
}

}  // namespace nsml
