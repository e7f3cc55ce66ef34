// Ordered stream compaction (Alg. 2 Steps 2-3: drop the pruned and the
// small-magnitude gradients, keep (index, value) of the rest in index order).
//
// One pass over the source.  Every element falls in one of three classes by
// its magnitude key: A (key >= hi) is always kept, C (lo <= key < hi) is kept
// while fewer than r class-C elements precede it in index order, the rest is
// dropped.  With r = "all" this writes a superset list for the later digit
// levels; with lo = T, hi = T+1 it applies the final threshold and tie budget.
//
// Tiles of kTile elements are handed out by an atomic ticket, so a tile's
// predecessors have always started.  Output offsets come from a chained scan
// over tiles (publish own counts, look back over predecessors until an
// inclusive prefix is found).  Every wait is bounded: when it runs out the
// block records NSML_ERR_TIMEOUT, marks its tile so that successors stop too,
// and leaves.
#pragma once

#include "nsml_common.cuh"

namespace nsml {

__device__ __forceinline__ unsigned long long pack_counts(unsigned long long a, unsigned long long c) {
  return (a << 31) | c;
}

__device__ __forceinline__ unsigned long long load_state(const unsigned long long* p) {
  return *reinterpret_cast<const volatile unsigned long long*>(p);
}

__device__ __forceinline__ void store_state(unsigned long long* p, unsigned long long v) {
  *reinterpret_cast<volatile unsigned long long*>(p) = v;
}

// Runs in warp 0 of the block that owns `tile`.  Returns the packed exclusive
// prefix (A << 31 | C) of the tile, or ~0 if the scan was abandoned.
__device__ unsigned long long chained_scan(unsigned long long* state, unsigned int tile,
                                           unsigned long long own, int* status) {
  const int lane = threadIdx.x & 31;
  if (tile == 0) {
    if (lane == 0) store_state(state, kFlagPrefix | own);
    return 0;
  }
  if (lane == 0) store_state(state + tile, kFlagAggregate | own);

  unsigned long long excl = 0;
  long long window_end = (long long)tile - 1;  // nearest predecessor of this window
  while (true) {
    const long long mine = window_end - lane;
    unsigned long long w = kFlagPrefix;  // tiles before 0 count as an empty prefix
    int polls = 0;
    bool gave_up = false;
    if (mine >= 0) {
      w = load_state(state + mine);
      while ((w & kFlagMask) == 0) {
        if (++polls > kMaxPolls) { gave_up = true; break; }
        __nanosleep(polls < 64 ? 20 : 400);
        w = load_state(state + mine);
      }
    }
    const unsigned int gave_up_mask = __ballot_sync(0xFFFFFFFFu, gave_up);
    const unsigned int abort_mask = __ballot_sync(0xFFFFFFFFu, (w & kFlagMask) == kFlagAbort);
    if (gave_up_mask | abort_mask) {
      if (lane == 0) {
        if (gave_up_mask) set_status(status, NSML_ERR_TIMEOUT);
        store_state(state + tile, kFlagAbort);
      }
      return ~0ull;
    }
    // nearest predecessor (lowest lane) that already holds an inclusive prefix
    const unsigned int has_prefix = __ballot_sync(0xFFFFFFFFu, (w & kFlagMask) == kFlagPrefix);
    const int stop = has_prefix ? (__ffs(has_prefix) - 1) : 32;
    unsigned long long contrib = (lane <= stop) ? (w & ~kFlagMask) : 0ull;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) contrib += __shfl_xor_sync(0xFFFFFFFFu, contrib, o);
    excl += contrib;
    if (has_prefix) break;
    window_end -= 32;
  }
  if (lane == 0) store_state(state + tile, kFlagPrefix | (excl + own));
  return excl;
}

// Compacts `count` elements of `src` into out_idx / out_val.  All threads of
// all blocks call this; returns when the ticket runs past the last tile.
template <class Src>
__device__ void compact_tiles(const Src& src, unsigned long long count, uint32_t lo, uint32_t hi,
                              unsigned long long r, unsigned int* ticket, unsigned long long* state,
                              int* status, uint32_t* __restrict__ out_idx, uint32_t* __restrict__ out_val,
                              unsigned long long* total_out) {
  __shared__ unsigned int s_tile;
  __shared__ unsigned int s_warp[kCta / 32];
  __shared__ unsigned long long s_excl;

  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;

  while (true) {
    __syncthreads();  // previous tile's shared values are no longer needed
    if (threadIdx.x == 0) s_tile = atomicAdd(ticket, 1u);
    __syncthreads();
    const unsigned int tile = s_tile;
    const unsigned long long base = (unsigned long long)tile * kTile;
    if (base >= count) return;

    // each warp owns 512 consecutive elements: 4 rounds of 32 lanes x 4
    Quad q[4];
    unsigned int fa[4], fc[4];      // per-round class flags, bit e = element e
    unsigned int excl_round[4];     // packed (A | C << 16) before this lane's quad, within the warp
    unsigned int running = 0;
#pragma unroll
    for (int j = 0; j < 4; ++j) q[j] = src.load4(base + warp * 512 + j * 128 + lane * 4, count);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      fa[j] = 0;
      fc[j] = 0;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const uint32_t key = q[j].bits[e] & 0x7FFFFFFFu;
        const bool v = (q[j].valid >> e) & 1u;
        const bool a = v && key >= hi;
        const bool c = v && !a && key >= lo;
        fa[j] |= (unsigned)a << e;
        fc[j] |= (unsigned)c << e;
      }
      const unsigned int mine = __popc(fa[j]) | (__popc(fc[j]) << 16);
      unsigned int incl = mine;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        unsigned int up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += up;
      }
      excl_round[j] = running + incl - mine;
      running += __shfl_sync(0xFFFFFFFFu, incl, 31);
    }
    if (lane == 0) s_warp[warp] = running;
    __syncthreads();

    unsigned int before_warp = 0, tile_total = 0;
#pragma unroll
    for (int w = 0; w < kCta / 32; ++w) {
      const unsigned int c = s_warp[w];
      if (w < warp) before_warp += c;
      tile_total += c;
    }

    if (warp == 0) {
      const unsigned long long own = pack_counts(tile_total & 0xFFFFu, tile_total >> 16);
      const unsigned long long e = chained_scan(state, tile, own, status);
      if (lane == 0) s_excl = e;
    }
    __syncthreads();
    const unsigned long long excl = s_excl;
    if (excl == ~0ull) return;  // abandoned: every thread of the block leaves

    const unsigned long long a0 = (excl >> 31) + (before_warp & 0xFFFFu);
    const unsigned long long c0 = (excl & kCountMask) + (before_warp >> 16);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if ((fa[j] | fc[j]) == 0) continue;
      unsigned long long a_before = a0 + (excl_round[j] & 0xFFFFu);
      unsigned long long c_before = c0 + (excl_round[j] >> 16);
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const bool a = (fa[j] >> e) & 1u;
        const bool c = (fc[j] >> e) & 1u;
        if (a || (c && c_before < r)) {
          const unsigned long long pos = a_before + (c_before < r ? c_before : r);
          out_idx[pos] = q[j].idx[e];
          out_val[pos] = q[j].bits[e];
        }
        a_before += a;
        c_before += c;
      }
    }

    if (base + kTile >= count && threadIdx.x == 0) {
      const unsigned long long a_all = (excl >> 31) + (tile_total & 0xFFFFu);
      const unsigned long long c_all = (excl & kCountMask) + (tile_total >> 16);
      *total_out = a_all + (c_all < r ? c_all : r);
    }
  }
}

// Bucket -> candidate list (superset of the survivors, or the survivors
// themselves when the threshold is already final).
template <int DTYPE>
__global__ void __launch_bounds__(kCta)
k_compact_bucket(BucketSrc<DTYPE> src, unsigned long long n, Ctl* ctl, unsigned long long* state,
                 uint32_t* list_idx, uint32_t* list_val) {
  compact_tiles(src, n, ctl->lo, ctl->hi, ctl->r, &ctl->ticket_bucket, state, &ctl->status,
                list_idx, list_val, &ctl->list_count);
}

// Candidate list -> final (index, raw value) arrays, applying the exact
// threshold key and tie budget.
__global__ void __launch_bounds__(kCta)
k_compact_list(ListSrc src, Ctl* ctl, unsigned long long* state, uint32_t* out_idx, uint32_t* out_val) {
  compact_tiles(src, ctl->list_count, ctl->lo, ctl->hi, ctl->r, &ctl->ticket_list, state, &ctl->status,
                out_idx, out_val, &ctl->out_count);
}

}  // namespace nsml
