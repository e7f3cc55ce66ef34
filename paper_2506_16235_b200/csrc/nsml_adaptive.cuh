// The steps of Alg. 2 around the top-k selection:
//   Step 1  the gradient's L2 norm for the adaptive-quantisation gate (k_sumsq)
//   Step 2  the pruning mask built from the weights: the ceil(0.5*(1-ratio)*n)
//           parameters of smallest magnitude, ties by lower index
//           (k_prune_hist, k_prune_ties, k_prune_write)
//   Step 3  "accumulate the local filtered gradients": the bucket that is
//           compressed is gradient + residual, and the residual keeps what the
//           payload does not carry (k_feedback_add, k_feedback_subtract)
// All of them stream the bucket with 16-byte loads, block-cyclically, so that
// the grid reads one moving window of memory.
#pragma once

#include "nsml_accumulate.cuh"
#include "nsml_codec.cuh"
#include "nsml_common.cuh"
#include "nsml_select.cuh"

namespace nsml {

constexpr int kStreamLoads = 4;  // 16-byte loads a thread keeps in flight
constexpr int kStreamTile = kCta * 4 * kStreamLoads;  // elements a block takes per step

// ------------------------------------------------------------------------
// Step 1: sum of squares in float64.  Every square is exact in float64 (a
// float32 has 24 significant bits), the adds follow a fixed order for a given
// grid (per thread, per warp, per block, then the last block to finish adds
// the per-block sums in block order), so the result is reproducible.
// ------------------------------------------------------------------------
struct SumsqCtl {
  int status;
  unsigned int ticket;  // blocks that have delivered their partial sum
  double sumsq;
};
constexpr int kSumsqMaxBlocks = 4096;
constexpr size_t kSumsqWorkspace = 256 + (size_t)kSumsqMaxBlocks * 8;

__device__ __forceinline__ double block_sum_f64(double t, double* s_red) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xFFFFFFFFu, t, o);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = t;
  __syncthreads();
  double b = 0.0;
#pragma unroll
  for (int w = 0; w < kCta / 32; ++w) b += s_red[w];
  return b;
}

template <int DTYPE>
__global__ void __launch_bounds__(kCta)
k_sumsq(BucketSrc<DTYPE> src, unsigned long long n, SumsqCtl* ctl, double* __restrict__ partials) {
  __shared__ double s_red[kCta / 32];
  __shared__ unsigned int s_last;
  const unsigned long long tiles = (n + kStreamTile - 1) / kStreamTile;
  double acc[4] = {0.0, 0.0, 0.0, 0.0};
  uint32_t worst = 0;  // largest magnitude key seen
  for (unsigned long long tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
    const unsigned long long base = tile * kStreamTile;
    uint32_t bits[kStreamLoads][4];
    if (base + kStreamTile <= n) {
#pragma unroll
      for (int u = 0; u < kStreamLoads; ++u) src.load_full4(base + (unsigned long long)(u * kCta + threadIdx.x) * 4, bits[u]);
    } else {
#pragma unroll
      for (int u = 0; u < kStreamLoads; ++u) src.load_vals4(base + (unsigned long long)(u * kCta + threadIdx.x) * 4, n, bits[u]);
    }
#pragma unroll
    for (int u = 0; u < kStreamLoads; ++u) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const double v = (double)__uint_as_float(bits[u][e]);
        acc[u & 3] = fma(v, v, acc[u & 3]);  // the product is exact, so this is one rounding, of the add
        worst = max(worst, bits[u][e] & 0x7FFFFFFFu);
      }
    }
  }
  if (worst >= kInfKey) set_status(&ctl->status, NSML_ERR_NONFINITE);
  const double block_total = block_sum_f64((acc[0] + acc[1]) + (acc[2] + acc[3]), s_red);
  if (threadIdx.x == 0) {
    partials[blockIdx.x] = block_total;
    __threadfence();
    s_last = atomicAdd(&ctl->ticket, 1u) == gridDim.x - 1;
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();  // the other blocks' partial sums are visible
  double p = 0.0;
  for (unsigned int i = threadIdx.x; i < gridDim.x; i += kCta) p += __ldcg(partials + i);
  const double total = block_sum_f64(p, s_red);
  if (threadIdx.x == 0) {
    ctl->sumsq = total;
    ctl->ticket = 0;
  }
}

// ------------------------------------------------------------------------
// Step 3, local accumulation.  residual <- gradient + residual (one float32
// add per element); the sum is what gets compressed.
// ------------------------------------------------------------------------
template <int DTYPE>
__global__ void __launch_bounds__(kCta)
k_feedback_add(BucketSrc<DTYPE> src, float* __restrict__ residual, unsigned long long n) {
  const unsigned long long tiles = (n + kStreamTile - 1) / kStreamTile;
  for (unsigned long long tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
    const unsigned long long base = tile * kStreamTile;
    if (base + kStreamTile <= n) {
      uint32_t g[kStreamLoads][4];
      float4 r[kStreamLoads];
#pragma unroll
      for (int u = 0; u < kStreamLoads; ++u) {
        const unsigned long long i0 = base + (unsigned long long)(u * kCta + threadIdx.x) * 4;
        src.load_full4(i0, g[u]);
        r[u] = *reinterpret_cast<const float4*>(residual + i0);
      }
#pragma unroll
      for (int u = 0; u < kStreamLoads; ++u) {
        const unsigned long long i0 = base + (unsigned long long)(u * kCta + threadIdx.x) * 4;
        float4 s;
        s.x = __fadd_rn(__uint_as_float(g[u][0]), r[u].x);
        s.y = __fadd_rn(__uint_as_float(g[u][1]), r[u].y);
        s.z = __fadd_rn(__uint_as_float(g[u][2]), r[u].z);
        s.w = __fadd_rn(__uint_as_float(g[u][3]), r[u].w);
        *reinterpret_cast<float4*>(residual + i0) = s;
      }
    } else {
      for (unsigned long long i = base + threadIdx.x; i < n; i += kCta)
        residual[i] = __fadd_rn(__uint_as_float(src.load1(i)), residual[i]);
    }
  }
}

// residual[idx_j] <- residual[idx_j] - v'_j for every payload entry, v' being the
// value a receiver reconstructs (one float32 subtraction).  Indices are unique,
// so entries do not interfere.
__global__ void __launch_bounds__(kCta)
k_feedback_subtract(const unsigned char* __restrict__ payload, float* __restrict__ residual, unsigned long long n,
                    int* status) {
  const nsml_payload_header* h = reinterpret_cast<const nsml_payload_header*>(payload);
  if (!header_ok(h, n)) {
    if (blockIdx.x == 0 && threadIdx.x == 0) set_status(status, NSML_ERR_PAYLOAD);
    return;
  }
  const unsigned long long k = h->k;
  const uint32_t* idx = reinterpret_cast<const uint32_t*>(payload + h->idx_off);
  const unsigned char* val = payload + h->val_off;
  const float* scale = reinterpret_cast<const float*>(payload + h->scale_off);
  const int bits = (int)h->bits;
  for (unsigned long long j = (unsigned long long)blockIdx.x * kCta + threadIdx.x; j < k;
       j += (unsigned long long)gridDim.x * kCta) {
    const uint32_t i = idx[j];
    float v;
    if (bits == NSML_BITS_INT8) v = decode_i8(reinterpret_cast<const signed char*>(val)[j], scale[j >> 10]);
    else if (bits == NSML_BITS_FP16) v = decode_f16(reinterpret_cast<const uint16_t*>(val)[j]);
    else v = reinterpret_cast<const float*>(val)[j];
    if (i < n) residual[i] = __fsub_rn(residual[i], v);
    else set_status(status, NSML_ERR_PAYLOAD);
  }
}

// ------------------------------------------------------------------------
// Step 2: pruning mask from the weights.  The m parameters of smallest
// magnitude, ties by lower index, are the m LARGEST under the complemented
// key (~bits & 0x7FFFFFFF) with the same tie rule, so this is the radix select
// of the top-k step on complemented keys: three histogram passes (12 + 12 + 7
// bits; each pass first resolves the previous level from the global
// histogram, every block for itself), an optional pass that counts the keys
// equal to the threshold per tile (needed only when not all of them are
// pruned), and the pass that writes the mask bits.
// ------------------------------------------------------------------------
struct PruneCtl {
  int status;
  unsigned int d0, rem1;       // digit 0 of the threshold, rank left inside its bin
  unsigned int prefix24, rem2; // digits 0-1, rank left
  unsigned int T, r, cT;       // threshold key (complemented), ties to prune, ties in all
  unsigned int list_count;     // entries appended to the tie list by the last histogram pass
  unsigned int list_ok;        // the tie list holds every key that shares the threshold's 24-bit prefix
  unsigned int use_limit;      // ties are decided by index: pruned iff index <= idx_limit
  unsigned int idx_limit;
  // two-pass path (sampled window)
  unsigned int win_lo, win_shift;  // window of complemented keys: bin = (key - win_lo) >> win_shift, kPruneFineBins bins
  unsigned int above;              // keys at or beyond the window's end
  unsigned int fast_ok;            // the window held the threshold and its bin was short enough to list: mask done in two passes
  unsigned int fast_bin, fast_rem; // the threshold's bin, rank left inside it
  unsigned int fast_listed;        // keys of that bin appended by the mask pass
};
constexpr int kPruneFineBins = 4096;
constexpr int kPruneSamples = 8192;
constexpr unsigned int kTieCap = 1024;  // keys sharing the threshold's 24-bit prefix that the tie list can hold

struct PruneLayout {
  size_t fine;       // u32[kPruneFineBins]: keys per bin of the sampled window (two-pass path)
  size_t hist;       // u32[3][kMaxBins]
  size_t tie_list;   // uint2[kTieCap]: (index, last key digit) of the keys that share the threshold's 24-bit prefix
  size_t tile_ties;  // u32[tiles]
  size_t total;
};

inline PruneLayout prune_layout(int64_t n) {
  PruneLayout L;
  const size_t tiles = ((size_t)n + kStreamTile - 1) / kStreamTile;
  L.fine = 256;
  L.hist = L.fine + kPruneFineBins * sizeof(unsigned int);
  L.tie_list = L.hist + 3 * kMaxBins * sizeof(unsigned int);
  L.tile_ties = L.tie_list + kTieCap * sizeof(uint2);
  L.total = L.tile_ties + align_up(tiles * 4, 256);
  return L;
}

__device__ __forceinline__ uint32_t prune_key(uint32_t bits) { return ~bits & 0x7FFFFFFFu; }

// Loads the block's share of one tile: bits[u][e] = element base + (u*kCta + t)*4 + e, cnt[u] of them exist.
__device__ __forceinline__ void load_tile(const BucketSrc<NSML_F32>& src, unsigned long long base, unsigned long long n,
                                          uint32_t (&bits)[kStreamLoads][4], int (&cnt)[kStreamLoads]) {
  if (base + kStreamTile <= n) {
#pragma unroll
    for (int u = 0; u < kStreamLoads; ++u) {
      src.load_full4(base + (unsigned long long)(u * kCta + threadIdx.x) * 4, bits[u]);
      cnt[u] = 4;
    }
  } else {
#pragma unroll
    for (int u = 0; u < kStreamLoads; ++u)
      cnt[u] = src.load_vals4(base + (unsigned long long)(u * kCta + threadIdx.x) * 4, n, bits[u]);
  }
}

// Resolves one level from its global histogram; every thread returns (digit, rank left).
template <int NB>
__device__ __forceinline__ void prune_resolve(const unsigned int* ghist, unsigned int rem, unsigned int* s_tot,
                                              unsigned int* s_out) {
  constexpr int PER = (NB + kCta - 1) / kCta;
  unsigned int own[PER];
#pragma unroll
  for (int b = 0; b < PER; ++b) {
    const int bin = threadIdx.x * PER + b;
    own[b] = (bin < NB) ? ghist[bin] : 0u;
  }
  find_digit_from_top<PER, kCta>(own, rem, s_tot, s_out);
}

template <int LEVEL>
__global__ void __launch_bounds__(kCta)
k_prune_hist(BucketSrc<NSML_F32> src, unsigned long long n, unsigned int m, PruneCtl* ctl, unsigned int* __restrict__ hist,
             uint2* __restrict__ tie_list) {
  constexpr int NB = (LEVEL == 2) ? 128 : kMaxBins;
  __shared__ unsigned int s_hist[NB];
  __shared__ unsigned int s_tot[kCta / 32], s_out[2];
  if (ctl->fast_ok != 0) return;  // the two-pass path has built the mask
  unsigned int prefix = 0;
  bool collect = false;
  // The block's first tile is requested before the previous level is resolved, so that the resolve (a read
  // of the 4096 global bins and a block-wide search) runs while those loads are in flight.
  const unsigned long long tiles = (n + kStreamTile - 1) / kStreamTile;
  uint32_t bits[kStreamLoads][4];
  bool preloaded = false;
  if (LEVEL != 0 && ((unsigned long long)blockIdx.x + 1) * kStreamTile <= n) {
#pragma unroll
    for (int u = 0; u < kStreamLoads; ++u)
      src.load_full4((unsigned long long)blockIdx.x * kStreamTile + (unsigned long long)(u * kCta + threadIdx.x) * 4, bits[u]);
    preloaded = true;
  }
  if (LEVEL == 1) {
    prune_resolve<kMaxBins>(hist, m, s_tot, s_out);
    prefix = s_out[0];
    if (blockIdx.x == 0 && threadIdx.x == 0) {
      ctl->d0 = s_out[0];
      ctl->rem1 = s_out[1];
    }
  } else if (LEVEL == 2) {
    prune_resolve<kMaxBins>(hist + kMaxBins, ctl->rem1, s_tot, s_out);
    prefix = (ctl->d0 << 12) | s_out[0];
    // Few keys share the threshold's first 24 bits (their number is the bin's count): this pass lists
    // them, so that ties at the threshold can be ranked by index without another pass over the weights.
    collect = hist[kMaxBins + s_out[0]] <= kTieCap;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
      ctl->prefix24 = prefix;
      ctl->rem2 = s_out[1];
      ctl->list_ok = collect;
    }
  }
  for (int b = threadIdx.x; b < NB; b += kCta) s_hist[b] = 0;
  __syncthreads();
  uint32_t lowest = 0x7FFFFFFFu;  // smallest complemented key seen: at most 0x007FFFFF for a NaN or an infinity
  // one key; (tile, u, e) locate it and are turned into an index only where one is needed
  auto visit = [&](uint32_t key, unsigned long long tile, int u, int e) {
    if (LEVEL == 0) {
      lowest = min(lowest, key);
      atomicAdd(&s_hist[key >> 19], 1u);
    } else if (LEVEL == 1) {
      if ((key >> 19) == prefix) atomicAdd(&s_hist[(key >> 7) & 0xFFFu], 1u);
    } else {
      if ((key >> 7) == prefix) {
        atomicAdd(&s_hist[key & 0x7Fu], 1u);
        if (collect) {
          const unsigned long long i = tile * kStreamTile + (unsigned long long)(u * kCta + threadIdx.x) * 4 + e;
          tie_list[atomicAdd(&ctl->list_count, 1u)] = make_uint2((uint32_t)i, key & 0x7Fu);
        }
      }
    }
  };
  for (unsigned long long tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
    const unsigned long long base = tile * kStreamTile;
    if (base + kStreamTile <= n) {  // a whole tile: no bounds checks
      if (!preloaded) {
#pragma unroll
        for (int u = 0; u < kStreamLoads; ++u) src.load_full4(base + (unsigned long long)(u * kCta + threadIdx.x) * 4, bits[u]);
      }
      preloaded = false;
#pragma unroll
      for (int u = 0; u < kStreamLoads; ++u)
#pragma unroll
        for (int e = 0; e < 4; ++e) visit(prune_key(bits[u][e]), tile, u, e);
    } else {
      int cnt[kStreamLoads];
#pragma unroll
      for (int u = 0; u < kStreamLoads; ++u)
        cnt[u] = src.load_vals4(base + (unsigned long long)(u * kCta + threadIdx.x) * 4, n, bits[u]);
#pragma unroll
      for (int u = 0; u < kStreamLoads; ++u)
#pragma unroll
        for (int e = 0; e < 4; ++e)
          if (e < cnt[u]) visit(prune_key(bits[u][e]), tile, u, e);
    }
  }
  const bool nonfinite = LEVEL == 0 && lowest <= 0x007FFFFFu;  // magnitude bits >= 0x7F800000
  if (nonfinite) set_status(&ctl->status, NSML_ERR_NONFINITE);
  __syncthreads();
  unsigned int* ghist = hist + LEVEL * kMaxBins;
  for (int b = threadIdx.x; b < NB; b += kCta) {
    const unsigned int c = s_hist[b];
    if (c) atomicAdd(&ghist[b], c);
  }
}

// Resolves the last digit: threshold T, ties to prune r, ties in all cT.  When r < cT only the r ties of
// lowest index are pruned.  Usually the last histogram pass has listed them: block 0 then finds the
// r-th smallest index among them and the mask pass compares indices with it.  Otherwise (more keys share
// the threshold's prefix than the list holds) the ties are counted per tile for a ranked mask pass.
__global__ void __launch_bounds__(kCta)
k_prune_ties(BucketSrc<NSML_F32> src, unsigned long long n, PruneCtl* ctl, const unsigned int* __restrict__ hist,
             const uint2* __restrict__ tie_list, unsigned int* __restrict__ tile_ties) {
  __shared__ unsigned int s_tot[kCta / 32], s_out[2];
  __shared__ unsigned int s_cnt[kCta / 32];
  __shared__ uint32_t s_tied[kTieCap];
  __shared__ unsigned int s_ntied;
  if (ctl->fast_ok != 0) return;  // the two-pass path has built the mask
  prune_resolve<128>(hist + 2 * kMaxBins, ctl->rem2, s_tot, s_out);
  const uint32_t T = (ctl->prefix24 << 7) | s_out[0];
  const unsigned int r = s_out[1], cT = hist[2 * kMaxBins + s_out[0]];
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    ctl->T = T;
    ctl->r = r;
    ctl->cT = cT;
  }
  if (r >= cT) return;  // every key equal to T is pruned: no ranks needed
  if (ctl->list_ok) {
    if (blockIdx.x != 0) return;
    if (threadIdx.x == 0) s_ntied = 0;
    __syncthreads();
    const unsigned int listed = min(ctl->list_count, kTieCap);
    for (unsigned int j = threadIdx.x; j < listed; j += kCta) {
      const uint2 e = tie_list[j];
      if (e.y == s_out[0]) s_tied[atomicAdd(&s_ntied, 1u)] = e.x;
    }
    __syncthreads();
    const unsigned int ntied = s_ntied;  // == cT
    for (unsigned int j = threadIdx.x; j < ntied; j += kCta) {
      const uint32_t mine = s_tied[j];
      unsigned int below = 0;
      for (unsigned int q = 0; q < ntied; ++q) below += s_tied[q] < mine;
      if (below == r - 1) {  // indices are distinct: exactly one entry has r - 1 below it
        ctl->idx_limit = mine;
        ctl->use_limit = 1;
      }
    }
    return;
  }
  const unsigned long long tiles = (n + kStreamTile - 1) / kStreamTile;
  for (unsigned long long tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
    uint32_t bits[kStreamLoads][4];
    int cnt[kStreamLoads];
    load_tile(src, tile * kStreamTile, n, bits, cnt);
    unsigned int c = 0;
#pragma unroll
    for (int u = 0; u < kStreamLoads; ++u)
#pragma unroll
      for (int e = 0; e < 4; ++e) c += (e < cnt[u]) && prune_key(bits[u][e]) == T;
    c = __reduce_add_sync(0xFFFFFFFFu, c);
    __syncthreads();  // s_cnt of the previous tile has been read
    if ((threadIdx.x & 31) == 0) s_cnt[threadIdx.x >> 5] = c;
    __syncthreads();
    if (threadIdx.x == 0) {
      unsigned int t = 0;
#pragma unroll
      for (int w = 0; w < kCta / 32; ++w) t += s_cnt[w];
      tile_ties[tile] = t;
    }
  }
}

// Writes the mask: bit (i & 31) of word i >> 5 set = parameter i pruned.  Bits past n in the last word are 0.
// Covers the two usual cases: every key equal to the threshold is pruned, or the ties are decided by index.
__global__ void __launch_bounds__(kCta)
k_prune_write(BucketSrc<NSML_F32> src, unsigned long long n, const PruneCtl* ctl, const unsigned int* __restrict__ tile_ties,
              uint32_t* __restrict__ mask) {
  if (ctl->fast_ok != 0) return;  // the two-pass path has built the mask
  const uint32_t T = ctl->T;
  const unsigned int r = ctl->r, cT = ctl->cT;
  const bool by_index = ctl->use_limit != 0;  // ties pruned iff their index is <= idx_limit
  const uint32_t idx_limit = ctl->idx_limit;
  const unsigned long long tiles = (n + kStreamTile - 1) / kStreamTile;
  const unsigned long long nwords = (n + 31) / 32;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  (void)tile_ties;
  if (r >= cT || by_index) {  // else: k_prune_write_ranked writes the mask
    // Every key > T is pruned, and every key == T (or, by_index, those up to idx_limit).  A warp's load
    // covers 128 consecutive elements = 4 mask words; the 4-bit
    // flags of 8 neighbouring lanes are combined into one word.
    // flags of this thread's four elements of load u -> the word shared by eight lanes
    auto word_of = [&](unsigned int f) {
      unsigned int x = f << (4 * (lane & 7));
      x |= __shfl_xor_sync(0xFFFFFFFFu, x, 1);
      x |= __shfl_xor_sync(0xFFFFFFFFu, x, 2);
      x |= __shfl_xor_sync(0xFFFFFFFFu, x, 4);
      return x;
    };
    auto is_pruned = [&](uint32_t key, unsigned long long base, int u, int e) {
      if (key == T)  // rare: the index is worked out only here (indices are below 2^31)
        return !by_index || (uint32_t)base + (uint32_t)((u * kCta + threadIdx.x) * 4 + e) <= idx_limit;
      return key > T;
    };
    // The same test on the weight itself: complemented key > T  <=>  |w| < tmag, key == T  <=>  |w| == tmag
    // (finite weights; denormals are not flushed), one compare with a free |.| instead of mask and compare.
    const float tmag = __uint_as_float(~T & 0x7FFFFFFFu);
    for (unsigned long long tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
      const unsigned long long base = tile * kStreamTile;
      uint32_t bits[kStreamLoads][4];
      uint32_t* out = mask + base / 32 + warp * 4 + (lane >> 3);  // word of load 0; load u is 32 words further
      if (base + kStreamTile <= n) {  // a whole tile: no bounds checks
#pragma unroll
        for (int u = 0; u < kStreamLoads; ++u) src.load_full4(base + (unsigned long long)(u * kCta + threadIdx.x) * 4, bits[u]);
#pragma unroll
        for (int u = 0; u < kStreamLoads; ++u) {
          unsigned int f = 0;
          bool tie = false;
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float a = fabsf(__uint_as_float(bits[u][e]));
            f |= (unsigned)(a < tmag) << e;
            tie |= a == tmag;
          }
          if (tie) {  // rare
            f = 0;
#pragma unroll
            for (int e = 0; e < 4; ++e) f |= (unsigned)is_pruned(prune_key(bits[u][e]), base, u, e) << e;
          }
          const unsigned int x = word_of(f);
          if ((lane & 7) == 0) out[u * (kCta / 8)] = x;
        }
      } else {
        int cnt[kStreamLoads];
#pragma unroll
        for (int u = 0; u < kStreamLoads; ++u)
          cnt[u] = src.load_vals4(base + (unsigned long long)(u * kCta + threadIdx.x) * 4, n, bits[u]);
#pragma unroll
        for (int u = 0; u < kStreamLoads; ++u) {
          unsigned int f = 0;
#pragma unroll
          for (int e = 0; e < 4; ++e) f |= (unsigned)((e < cnt[u]) && is_pruned(prune_key(bits[u][e]), base, u, e)) << e;
          const unsigned int x = word_of(f);
          const unsigned long long word = base / 32 + warp * 4 + (lane >> 3) + (unsigned long long)u * (kCta / 8);
          if ((lane & 7) == 0 && word < nwords) mask[word] = x;
        }
      }
    }
  }
}

// The mask pass for the remaining case: some of the keys equal to T stay unpruned and there are too many
// of them to list, so the first r of them in index order are found by rank.  Returns at once otherwise.
__global__ void __launch_bounds__(kCta)
k_prune_write_ranked(BucketSrc<NSML_F32> src, unsigned long long n, const PruneCtl* ctl,
                     const unsigned int* __restrict__ tile_ties, uint32_t* __restrict__ mask) {
  __shared__ unsigned int s_scan[kCta / 32];
  __shared__ unsigned long long s_red[kCta / 32];
  const uint32_t T = ctl->T;
  const unsigned int r = ctl->r, cT = ctl->cT;
  if (ctl->fast_ok != 0 || r >= cT || ctl->use_limit != 0) return;
  const unsigned long long tiles = (n + kStreamTile - 1) / kStreamTile;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  // A block takes a contiguous range of tiles and carries the number of ties seen so far; within a tile a thread
  // owns one mask word (32 consecutive elements).
  const unsigned long long t_first = (unsigned long long)blockIdx.x * tiles / gridDim.x;
  const unsigned long long t_last = (unsigned long long)(blockIdx.x + 1) * tiles / gridDim.x;
  unsigned long long before = 0;
  for (unsigned long long t = threadIdx.x; t < t_first; t += kCta) before += tile_ties[t];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) before += __shfl_xor_sync(0xFFFFFFFFu, before, o);
  if (lane == 0) s_red[warp] = before;
  __syncthreads();
  before = 0;
#pragma unroll
  for (int w = 0; w < kCta / 32; ++w) before += s_red[w];
  constexpr int kWordsPerTile = kStreamTile / 32;  // a thread owns one word of the tile
  static_assert(kWordsPerTile <= kCta, "one mask word per thread");
  for (unsigned long long tile = t_first; tile < t_last; ++tile) {
    const unsigned long long i0 = tile * kStreamTile + (unsigned long long)threadIdx.x * 32;
    uint32_t key[32];
    unsigned int ties = 0;
    const bool owner = threadIdx.x < kWordsPerTile && i0 < n;
    if (owner) {
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        uint32_t b4[4];
        const int c = src.load_vals4(i0 + q * 4, n, b4);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          key[q * 4 + e] = (e < c) ? prune_key(b4[e]) : 0u;  // key 0 = missing (a real key 0 would be NaN)
          ties += (e < c) && key[q * 4 + e] == T;
        }
      }
    }
    // exclusive scan of the per-thread tie counts over the block
    unsigned int incl = ties;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned int up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
      if (lane >= o) incl += up;
    }
    __syncthreads();  // s_scan of the previous tile has been read
    if (lane == 31) s_scan[warp] = incl;
    __syncthreads();
    unsigned int warps_before = 0, all = 0;
#pragma unroll
    for (int w = 0; w < kCta / 32; ++w) {
      const unsigned int c = s_scan[w];
      if (w < warp) warps_before += c;
      all += c;
    }
    if (owner) {
      unsigned long long rank = before + warps_before + incl - ties;
      uint32_t word = 0;
#pragma unroll
      for (int e = 0; e < 32; ++e) {
        const bool tie = key[e] == T && T != 0u;
        const bool pruned = key[e] > T || (tie && rank < r);
        rank += tie;
        word |= (uint32_t)pruned << e;
      }
      mask[i0 / 32] = word;
    }
    before += all;
  }
}

// ------------------------------------------------------------------------
// Step 2 in two passes over the weights instead of four.  A stratified sample
// of the weights brackets the m-th largest complemented key between two sample
// keys six sigma apart (k_prune_sample); one pass counts the keys beyond the
// bracket and the keys inside it in kPruneFineBins bins (k_prune_count); one
// block finds the bin that holds the threshold (k_prune_settle); the mask pass
// prunes everything beyond that bin and lists the bin's few keys
// (k_prune_mark); one block ranks the listed keys - larger complemented key
// first, then lower index - and sets the bits of the first `rem` of them
// (k_prune_fix).  When the sample misleads (the threshold lies outside the
// bracket) or the bin holds more keys than can be listed (massive ties),
// fast_ok stays 0 and the four-pass kernels above, which are enqueued behind
// these in any case and otherwise leave at once, build the mask: the result is
// exact either way.
// ------------------------------------------------------------------------
__global__ void __launch_bounds__(1024)
k_prune_sample(BucketSrc<NSML_F32> src, unsigned long long n, unsigned int rank_lo, unsigned int rank_hi, PruneCtl* ctl) {
  constexpr int THREADS = 1024, PER_THREAD = kPruneSamples / THREADS;  // 8 scattered loads in flight per thread
  __shared__ __align__(16) unsigned int s_hist_lo[kMaxBins];
  __shared__ __align__(16) unsigned int s_hist_hi[kMaxBins];
  __shared__ unsigned int s_tot[THREADS / 32], s_out[2];
  const int t = threadIdx.x;
  const unsigned long long width = n / kPruneSamples;  // >= 2
  uint32_t keys[PER_THREAD];
#pragma unroll
  for (int s = 0; s < PER_THREAD; ++s) {
    const unsigned int stratum = (unsigned int)s * THREADS + t;
    const unsigned long long pos = (unsigned long long)stratum * width +
                                   (((unsigned long long)mix32(stratum * 0x9E3779B1u + 0x85EBCA6Bu) * width) >> 32);
    keys[s] = prune_key(src.raw1(pos));
  }
  unsigned int prefix_lo = 0, prefix_hi = 0, rem_lo = rank_lo, rem_hi = rank_hi;
#pragma unroll
  for (int level = 0; level < 2; ++level) {  // 12 + 12 bits
    const int shift = digit_shift(level);
    __syncthreads();
    for (int b = t; b < kMaxBins; b += THREADS) {
      s_hist_lo[b] = 0;
      s_hist_hi[b] = 0;
    }
    __syncthreads();
#pragma unroll
    for (int s = 0; s < PER_THREAD; ++s) {
      const unsigned int bin = (keys[s] >> shift) & (kMaxBins - 1);
      if (level == 0 || (keys[s] >> 19) == prefix_lo) atomicAdd(&s_hist_lo[bin], 1u);
      if (level == 1 && (keys[s] >> 19) == prefix_hi) atomicAdd(&s_hist_hi[bin], 1u);
    }
    __syncthreads();
    unsigned int own[4];
    {
      const uint4 v = reinterpret_cast<const uint4*>(s_hist_lo)[t];
      own[0] = v.x; own[1] = v.y; own[2] = v.z; own[3] = v.w;
    }
    find_digit_from_top<4, THREADS>(own, rem_lo, s_tot, s_out);
    prefix_lo = (prefix_lo << 12) | s_out[0];
    rem_lo = s_out[1];
    if (level == 1) {
      const uint4 h = reinterpret_cast<const uint4*>(s_hist_hi)[t];
      own[0] = h.x; own[1] = h.y; own[2] = h.z; own[3] = h.w;
    }
    find_digit_from_top<4, THREADS>(own, rem_hi, s_tot, s_out);
    prefix_hi = (prefix_hi << 12) | s_out[0];
    rem_hi = s_out[1];
  }
  if (t != 0) return;
  const unsigned int lo = prefix_lo << 7, hi = (prefix_hi + 1u) << 7;  // hi: first key above hi's 24-bit class
  const unsigned int span = hi > lo ? hi - lo : 0u;
  unsigned int shift = 0;
  while ((span >> shift) >= (unsigned int)(kPruneFineBins * 3 / 4)) ++shift;
  ctl->win_lo = lo;
  ctl->win_shift = shift;
}

// Pass 1: keys beyond the window are counted, keys inside it (about 7 % of them) go into the block's copy of the
// window's histogram in shared memory, which is added to the global one at the end (a warp's adds go to 32
// neighbouring counters, one memory transaction; single adds to scattered counters run at a few dozen per ns for
// the whole GPU and made this pass 85 us).
__global__ void __launch_bounds__(kCta)
k_prune_count(BucketSrc<NSML_F32> src, unsigned long long n, PruneCtl* ctl, unsigned int* __restrict__ fine) {
  __shared__ unsigned int s_hist[kPruneFineBins];
  __shared__ unsigned int s_above[kCta / 32];
  const unsigned int lo = ctl->win_lo, shift = ctl->win_shift;
  for (int b = threadIdx.x; b < kPruneFineBins; b += kCta) s_hist[b] = 0;
  __syncthreads();
  const unsigned long long tiles = (n + kStreamTile - 1) / kStreamTile;
  // The tests run on the weight itself: complemented key >= E  <=>  |w| <= float(0x7FFFFFFF - E) for finite w.
  const unsigned long long win_end = (unsigned long long)lo + ((unsigned long long)kPruneFineBins << shift);
  const float t_end = win_end > 0x7FFFFFFFull ? -1.0f : __uint_as_float(min(0x7FFFFFFFu - (unsigned int)win_end, 0x7F7FFFFFu));
  const float t_lo = __uint_as_float(min(0x7FFFFFFFu - lo, 0x7F7FFFFFu));
  unsigned int above = 0;
  bool nonfinite = false;
  for (unsigned long long tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
    uint32_t bits[kStreamLoads][4];
    int cnt[kStreamLoads];
    const bool whole = (tile + 1) * kStreamTile <= n;
    load_tile(src, tile * kStreamTile, n, bits, cnt);
#pragma unroll
    for (int u = 0; u < kStreamLoads; ++u)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        if (!whole && e >= cnt[u]) continue;
        const float a = fabsf(__uint_as_float(bits[u][e]));
        nonfinite |= !(a <= 3.4028234663852886e38f);  // NaN or an infinity
        const bool beyond = a <= t_end;
        above += beyond;
        if (!beyond && a <= t_lo) atomicAdd(&s_hist[(prune_key(bits[u][e]) - lo) >> shift], 1u);  // about 7 % of the keys
      }
  }
  if (nonfinite) set_status(&ctl->status, NSML_ERR_NONFINITE);
  above = __reduce_add_sync(0xFFFFFFFFu, above);
  if ((threadIdx.x & 31) == 0) s_above[threadIdx.x >> 5] = above;
  __syncthreads();
  for (int b = threadIdx.x; b < kPruneFineBins; b += kCta) {
    const unsigned int c = s_hist[b];
    if (c != 0) atomicAdd(fine + b, c);  // result unused: a reduction
  }
  if (threadIdx.x == 0) {
    unsigned int t = 0;
#pragma unroll
    for (int w = 0; w < kCta / 32; ++w) t += s_above[w];
    if (t != 0) atomicAdd(&ctl->above, t);
  }
}

// One block: the window's bin that holds the m-th largest key, if the window holds it at all.
__global__ void __launch_bounds__(kCta)
k_prune_settle(unsigned int m, PruneCtl* ctl, const unsigned int* __restrict__ fine) {
  __shared__ unsigned int s_tot[kCta / 32], s_out[2];
  __shared__ unsigned long long s_sum[kCta / 32];
  constexpr int PER = kPruneFineBins / kCta;
  unsigned int own[PER];
  unsigned long long mine = 0;
#pragma unroll
  for (int b = 0; b < PER; ++b) {
    own[b] = __ldcg(fine + threadIdx.x * PER + b);
    mine += own[b];
  }
  const unsigned int above = __ldcg(&ctl->above);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mine += __shfl_xor_sync(0xFFFFFFFFu, mine, o);
  if ((threadIdx.x & 31) == 0) s_sum[threadIdx.x >> 5] = mine;
  __syncthreads();
  unsigned long long inside = 0;
#pragma unroll
  for (int w = 0; w < kCta / 32; ++w) inside += s_sum[w];
  if (m <= above || (unsigned long long)m > above + inside) return;  // the threshold lies outside the window
  find_digit_from_top<PER, kCta>(own, m - above, s_tot, s_out);
  if (threadIdx.x == 0) {
    const unsigned int bin = s_out[0];
    if (__ldcg(fine + bin) <= kTieCap) {  // short enough to list
      ctl->fast_bin = bin;
      ctl->fast_rem = s_out[1];
      ctl->fast_ok = 1u;
    }
  }
}

// Pass 2: prunes every key beyond the threshold's bin, lists the bin's keys (their bits stay 0 for k_prune_fix).
// The tests run on the weight itself: complemented key >= E  <=>  |w| <= float(0x7FFFFFFF - E) for finite w.
__global__ void __launch_bounds__(kCta)
k_prune_mark(BucketSrc<NSML_F32> src, unsigned long long n, PruneCtl* ctl, uint2* __restrict__ tie_list,
             uint32_t* __restrict__ mask) {
  if (ctl->fast_ok == 0) return;
  const unsigned long long bin_lo = (unsigned long long)ctl->win_lo + ((unsigned long long)ctl->fast_bin << ctl->win_shift);
  const unsigned long long bin_hi = bin_lo + (1ull << ctl->win_shift);  // first key beyond the bin
  // largest magnitude key that is pruned for sure / that is still in the bin (0x7F7FFFFF: the largest finite)
  const float t_beyond = bin_hi > 0x7FFFFFFFull ? -1.0f : __uint_as_float(min(0x7FFFFFFFu - (unsigned int)bin_hi, 0x7F7FFFFFu));
  const float t_bin = __uint_as_float(min(0x7FFFFFFFu - (unsigned int)bin_lo, 0x7F7FFFFFu));
  const unsigned long long tiles = (n + kStreamTile - 1) / kStreamTile;
  const unsigned long long nwords = (n + 31) / 32;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (unsigned long long tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
    const unsigned long long base = tile * kStreamTile;
    uint32_t bits[kStreamLoads][4];
    int cnt[kStreamLoads];
    const bool whole = base + kStreamTile <= n;
    load_tile(src, base, n, bits, cnt);
#pragma unroll
    for (int u = 0; u < kStreamLoads; ++u) {
      unsigned int f = 0;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        if (!whole && e >= cnt[u]) continue;
        const float a = fabsf(__uint_as_float(bits[u][e]));
        if (a <= t_beyond) {
          f |= 1u << e;
        } else if (a <= t_bin) {  // rare: at most kTieCap keys in the whole bucket
          const unsigned int slot = atomicAdd(&ctl->fast_listed, 1u);
          const unsigned long long i = base + (unsigned long long)(u * kCta + threadIdx.x) * 4 + e;
          if (slot < kTieCap) tie_list[slot] = make_uint2((uint32_t)i, prune_key(bits[u][e]));
        }
      }
      // the 4-bit flags of eight neighbouring lanes make one mask word
      unsigned int x = f << (4 * (lane & 7));
      x |= __shfl_xor_sync(0xFFFFFFFFu, x, 1);
      x |= __shfl_xor_sync(0xFFFFFFFFu, x, 2);
      x |= __shfl_xor_sync(0xFFFFFFFFu, x, 4);
      const unsigned long long word = base / 32 + warp * 4 + (lane >> 3) + (unsigned long long)u * (kCta / 8);
      if ((lane & 7) == 0 && word < nwords) mask[word] = x;
    }
  }
}

// The first fast_rem of the listed keys under (complemented key descending, index ascending) are pruned.  Every
// block holds the whole list and ranks its share of the entries (ranking is quadratic in the list's length).
constexpr int kPruneFixBlocks = 16;
__global__ void __launch_bounds__(kCta)
k_prune_fix(PruneCtl* ctl, const uint2* __restrict__ tie_list, uint32_t* __restrict__ mask) {
  __shared__ uint2 s_list[kTieCap];
  if (ctl->fast_ok == 0) return;
  const unsigned int listed = min(__ldcg(&ctl->fast_listed), kTieCap), rem = ctl->fast_rem;
  for (unsigned int i = threadIdx.x; i < listed; i += kCta) s_list[i] = __ldcg(tie_list + i);
  __syncthreads();
  if (listed < rem) {  // cannot happen: the bin holds at least rem keys
    if (threadIdx.x == 0) set_status(&ctl->status, NSML_ERR_INTERNAL);
    return;
  }
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  // a warp per entry, the lanes share the comparisons
  for (unsigned int i = blockIdx.x * (kCta / 32) + warp; i < listed; i += gridDim.x * (kCta / 32)) {
    const uint2 me = s_list[i];
    unsigned int before = 0;
    for (unsigned int q = lane; q < listed; q += 32) {
      const uint2 e = s_list[q];
      before += e.y > me.y || (e.y == me.y && e.x < me.x);
    }
    before = __reduce_add_sync(0xFFFFFFFFu, before);
    if (lane == 0 && before < rem) atomicOr(mask + (me.x >> 5), 1u << (me.x & 31));
  }
}

}  // namespace nsml
