// Candidate list -> payload, in one cooperative kernel.
//
// The bucket pass leaves a segmented list of candidates (every key >= lo).
// This kernel finds the exact threshold key T and the tie budget r by radix
// select on the candidates' magnitude keys (12 + 12 + 7 bits, Alg. 2 Step 3
// read as: keep the k largest |g|, ties by lower index), writes the k
// survivors in index order and quantises them (Alg. 2 Step 1 "quantize" for
// fp16; int8 per block of 1024 survivors).
//
// All blocks are co-resident (cooperative launch); block b owns a contiguous
// run of segments, i.e. a contiguous index range, for the whole kernel, so
// "index order" is block order.  Phases are separated by grid barriers:
//   1  count own candidates, histogram of key digit 0        | barrier
//   2  every block resolves digit 0; histogram of digit 1    | barrier
//   3  resolve digit 1; histogram of digit 2                 | barrier
//   4  resolve digit 2 -> T, r; count own (> T, == T)        | barrier
//   5  prefix over blocks; write survivors (index, value)    | barrier
//   6  quantise blocks of 1024 survivors, write the header
// If the list holds fewer than k candidates (fewer than k non-zero keys, or a
// misleading sample) phase 1 is followed by a slow path that rebuilds the
// segments from the bucket: every non-zero key plus the first k - nnz zeros in
// index order; then phase 1 runs again.
//
// Every barrier wait is bounded: when it runs out the block records
// NSML_ERR_TIMEOUT and leaves; the others then time out as well.
#pragma once

#include "nsml_codec.cuh"
#include "nsml_common.cuh"
#include "nsml_compact.cuh"
#include "nsml_select.cuh"

namespace nsml {

constexpr int kMaxSegPerBlock = 64;

struct FinalizeParams {
  unsigned long long n, k;
  int bits;
  unsigned int segments;             // warps of the bucket pass
  Ctl* ctl;
  unsigned int* hist;                // [4][kMaxBins]
  unsigned long long* block_counts;  // [4][kMaxFinalizeBlocks]
  unsigned int* seg_count;
  unsigned int* seg_zeros;
  uint32_t* seg_idx;
  uint32_t* seg_val;
  float* raw_val;
  unsigned char* payload;
  PayloadLayout P;
};

struct FinalizeShared {
  unsigned int hist[kMaxBins];
  unsigned long long red[kCta / 32];
  unsigned int tot[kCta / 32];
  unsigned int out[2];
  unsigned int seg_a[kMaxSegPerBlock];
  unsigned int seg_c[kMaxSegPerBlock];
  float qmax[kCta / 32];
  int ok;
};

__device__ __forceinline__ unsigned long long ld_cg_u64(const unsigned long long* p) {
  return __ldcg(p);
}

// Sum over the block; every thread gets the result.
__device__ __forceinline__ unsigned long long block_sum(unsigned long long v, FinalizeShared& sh) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) sh.red[threadIdx.x >> 5] = v;
  __syncthreads();
  unsigned long long s = 0;
#pragma unroll
  for (int w = 0; w < kCta / 32; ++w) s += sh.red[w];
  return s;
}

// All blocks arrive, then all leave.  `target` = barrier ordinal * gridDim.x.
__device__ __forceinline__ bool grid_barrier(Ctl* ctl, unsigned int target, FinalizeShared& sh) {
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    atomicAdd(&ctl->barrier, 1u);
    int ok = 1, polls = 0;
    while (*reinterpret_cast<volatile unsigned int*>(&ctl->barrier) < target) {
      if (++polls > kMaxPolls) { ok = 0; break; }
      if (polls > 64) __nanosleep(100);
    }
    __threadfence();
    if (!ok) set_status(&ctl->status, NSML_ERR_TIMEOUT);
    sh.ok = ok;
  }
  __syncthreads();
  return sh.ok != 0;
}

// Adds the block's shared histogram into the global one (non-empty bins only).
template <int NB>
__device__ __forceinline__ void flush_hist(FinalizeShared& sh, unsigned int* ghist) {
  __syncthreads();
  for (int b = threadIdx.x; b < NB; b += kCta) {
    const unsigned int c = sh.hist[b];
    if (c) atomicAdd(&ghist[b], c);
  }
}

// Every block reads the global histogram of a level and finds the digit that
// holds the rem-th largest key; returns it and the rank left inside (sh.out).
template <int NB>
__device__ __forceinline__ void resolve_digit(const unsigned int* ghist, unsigned int rem, FinalizeShared& sh) {
  constexpr int PER = (NB + kCta - 1) / kCta;
  unsigned int own[PER];
#pragma unroll
  for (int b = 0; b < PER; ++b) {
    const int bin = threadIdx.x * PER + b;
    own[b] = (bin < NB) ? __ldcg(ghist + bin) : 0u;
  }
  find_digit_from_top<PER, kCta>(own, rem, sh.tot, sh.out);
}

template <int DTYPE>
__global__ void __launch_bounds__(kCta, 4)
k_finalize(BucketSrc<DTYPE> src, FinalizeParams p) {
  __shared__ FinalizeShared sh;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const unsigned int G = gridDim.x, blk = blockIdx.x;
  const unsigned int s0 = (unsigned int)((unsigned long long)blk * p.segments / G);
  const unsigned int s1 = (unsigned int)((unsigned long long)(blk + 1) * p.segments / G);
  const unsigned long long rounds = (p.n + kRound - 1) / kRound;
  unsigned int barriers = 0;
  unsigned long long list_total = 0;
  int used_attempt = 0;  // which level-0 histogram belongs to the list in use

  // ---------------- phase 1 (twice if the slow path runs) ----------------
  for (int attempt = 0; attempt < 2; ++attempt) {
    unsigned int* ghist0 = p.hist + (attempt == 0 ? 0 : 3) * kMaxBins;
    unsigned long long* totals = p.block_counts + (attempt == 0 ? 0 : 3) * kMaxFinalizeBlocks;
    for (int b = threadIdx.x; b < kMaxBins; b += kCta) sh.hist[b] = 0;
    __syncthreads();
    unsigned long long mine = 0;
    bool nonfinite = false;
    for (unsigned int seg = s0 + warp; seg < s1; seg += kCta / 32) {
      const unsigned int cnt = __ldcg(p.seg_count + seg);
      const unsigned long long base = warp_first_round(seg, p.segments, rounds) * kRound;
      for (unsigned int i = lane; i < cnt; i += 32) {
        const uint32_t key = __ldcg(p.seg_val + base + i) & 0x7FFFFFFFu;
        nonfinite |= key >= kInfKey;
        atomicAdd(&sh.hist[key >> digit_shift(0)], 1u);
      }
      if (lane == 0) mine += cnt;
    }
    if (nonfinite) set_status(&p.ctl->status, NSML_ERR_NONFINITE);
    const unsigned long long block_total = block_sum(mine, sh);
    if (threadIdx.x == 0) totals[blk] = block_total;
    flush_hist<kMaxBins>(sh, ghist0);
    if (!grid_barrier(p.ctl, ++barriers * G, sh)) return;

    unsigned long long part = 0;
    for (unsigned int b = threadIdx.x; b < G; b += kCta) part += ld_cg_u64(totals + b);
    list_total = block_sum(part, sh);
    used_attempt = attempt;
    if (list_total >= p.k) break;
    if (attempt == 1) {  // cannot happen: the rebuilt list holds at least k entries
      if (threadIdx.x == 0) set_status(&p.ctl->status, NSML_ERR_INTERNAL);
      return;
    }

    // ---- slow path: rebuild own segments as (all non-zero keys) + (zeros within budget) ----
    unsigned long long nnz = 0, zeros = 0;
    for (unsigned int seg = s0 + warp; seg < s1; seg += kCta / 32) {
      const unsigned long long first = warp_first_round(seg, p.segments, rounds);
      const unsigned long long last = warp_first_round(seg + 1ull, p.segments, rounds);
      unsigned int seg_nnz = 0, seg_zero = 0;
      for (unsigned long long rd = first; rd < last; ++rd) {
        uint32_t bits[4];
        const int cnt = src.load_vals4(rd * kRound + lane * 4, p.n, bits);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          if (e < cnt) {
            if ((bits[e] & 0x7FFFFFFFu) != 0) ++seg_nnz; else ++seg_zero;
          }
        }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        seg_nnz += __shfl_xor_sync(0xFFFFFFFFu, seg_nnz, o);
        seg_zero += __shfl_xor_sync(0xFFFFFFFFu, seg_zero, o);
      }
      if (lane == 0) {
        p.seg_zeros[seg] = seg_zero;
        nnz += seg_nnz;
        zeros += seg_zero;
      }
    }
    const unsigned long long block_nnz = block_sum(nnz, sh);
    const unsigned long long block_zeros = block_sum(zeros, sh);
    unsigned long long* nz_counts = p.block_counts + 2 * kMaxFinalizeBlocks;
    if (threadIdx.x == 0) nz_counts[blk] = (block_nnz << 32) | block_zeros;
    if (!grid_barrier(p.ctl, ++barriers * G, sh)) return;

    unsigned long long all_nnz = 0, zeros_before = 0;
    for (unsigned int b = threadIdx.x; b < G; b += kCta) {
      const unsigned long long w = ld_cg_u64(nz_counts + b);
      all_nnz += w >> 32;
      if (b < blk) zeros_before += w & 0xFFFFFFFFull;
    }
    all_nnz = block_sum(all_nnz, sh);
    zeros_before = block_sum(zeros_before, sh);
    const unsigned long long zero_budget = (p.k > all_nnz) ? p.k - all_nnz : 0;

    for (unsigned int seg = s0 + warp; seg < s1; seg += kCta / 32) {
      unsigned long long before = zeros_before;
      for (unsigned int s = s0; s < seg; ++s) before += __ldcg(p.seg_zeros + s);
      const unsigned long long seg_zero = __ldcg(p.seg_zeros + seg);
      const unsigned long long allowed =
          (zero_budget > before) ? min(seg_zero, zero_budget - before) : 0ull;  // zeros of this segment to keep
      const unsigned long long first = warp_first_round(seg, p.segments, rounds);
      const unsigned long long last = warp_first_round(seg + 1ull, p.segments, rounds);
      const unsigned long long seg_base = first * kRound;
      unsigned int kept = 0, zeros_seen = 0;
      for (unsigned long long rd = first; rd < last; ++rd) {
        uint32_t bits[4];
        const int cnt = src.load_vals4(rd * kRound + lane * 4, p.n, bits);
        unsigned int fz = 0, fn = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          if (e < cnt) {
            if ((bits[e] & 0x7FFFFFFFu) != 0) fn |= 1u << e; else fz |= 1u << e;
          }
        }
        // zeros before this lane's quad in the round, then which of its zeros are within budget
        const unsigned int zmine = __popc(fz);
        unsigned int zincl = zmine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const unsigned int up = __shfl_up_sync(0xFFFFFFFFu, zincl, o);
          if (lane >= o) zincl += up;
        }
        unsigned long long zrank = zeros_seen + zincl - zmine;
        unsigned int f = fn;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          if (fz & (1u << e)) {
            if (zrank < allowed) f |= 1u << e;
            ++zrank;
          }
        }
        zeros_seen += __shfl_sync(0xFFFFFFFFu, zincl, 31);
        if (__any_sync(0xFFFFFFFFu, f != 0))
          kept += append_round(f, bits, (uint32_t)(rd * kRound), seg_base + kept, p.seg_idx, p.seg_val);
      }
      if (lane == 0) p.seg_count[seg] = kept;
    }
    __threadfence();
    __syncthreads();
  }

  const unsigned int* ghist0_final = p.hist + (used_attempt == 0 ? 0 : 3) * kMaxBins;

  // ---------------- phase 2: resolve digit 0, histogram of digit 1 ----------------
  resolve_digit<kMaxBins>(ghist0_final, (unsigned int)p.k, sh);
  const unsigned int d0 = sh.out[0];
  unsigned int rem = sh.out[1];
  for (int b = threadIdx.x; b < kMaxBins; b += kCta) sh.hist[b] = 0;
  __syncthreads();
  for (unsigned int seg = s0 + warp; seg < s1; seg += kCta / 32) {
    const unsigned int cnt = __ldcg(p.seg_count + seg);
    const unsigned long long base = warp_first_round(seg, p.segments, rounds) * kRound;
    for (unsigned int i = lane; i < cnt; i += 32) {
      const uint32_t key = __ldcg(p.seg_val + base + i) & 0x7FFFFFFFu;
      if ((key >> 19) == d0) atomicAdd(&sh.hist[(key >> 7) & 0xFFFu], 1u);
    }
  }
  flush_hist<kMaxBins>(sh, p.hist + 1 * kMaxBins);
  if (!grid_barrier(p.ctl, ++barriers * G, sh)) return;

  // ---------------- phase 3: resolve digit 1, histogram of digit 2 ----------------
  resolve_digit<kMaxBins>(p.hist + 1 * kMaxBins, rem, sh);
  const unsigned int prefix24 = (d0 << 12) | sh.out[0];
  rem = sh.out[1];
  for (int b = threadIdx.x; b < 128; b += kCta) sh.hist[b] = 0;
  __syncthreads();
  for (unsigned int seg = s0 + warp; seg < s1; seg += kCta / 32) {
    const unsigned int cnt = __ldcg(p.seg_count + seg);
    const unsigned long long base = warp_first_round(seg, p.segments, rounds) * kRound;
    for (unsigned int i = lane; i < cnt; i += 32) {
      const uint32_t key = __ldcg(p.seg_val + base + i) & 0x7FFFFFFFu;
      if ((key >> 7) == prefix24) atomicAdd(&sh.hist[key & 0x7Fu], 1u);
    }
  }
  flush_hist<128>(sh, p.hist + 2 * kMaxBins);
  if (!grid_barrier(p.ctl, ++barriers * G, sh)) return;

  // ---------------- phase 4: T and r; count own keys > T and == T ----------------
  resolve_digit<128>(p.hist + 2 * kMaxBins, rem, sh);
  const uint32_t T = (prefix24 << 7) | sh.out[0];
  const unsigned long long r = sh.out[1];  // ties (key == T) to keep, lowest index first
  unsigned long long mine_a = 0, mine_c = 0;
  for (unsigned int seg = s0 + warp; seg < s1; seg += kCta / 32) {
    const unsigned int cnt = __ldcg(p.seg_count + seg);
    const unsigned long long base = warp_first_round(seg, p.segments, rounds) * kRound;
    unsigned int a = 0, c = 0;
    for (unsigned int i = lane; i < cnt; i += 32) {
      const uint32_t key = __ldcg(p.seg_val + base + i) & 0x7FFFFFFFu;
      a += key > T;
      c += key == T;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      a += __shfl_xor_sync(0xFFFFFFFFu, a, o);
      c += __shfl_xor_sync(0xFFFFFFFFu, c, o);
    }
    if (lane == 0) {
      sh.seg_a[seg - s0] = a;
      sh.seg_c[seg - s0] = c;
      mine_a += a;
      mine_c += c;
    }
  }
  const unsigned long long block_a = block_sum(mine_a, sh);
  const unsigned long long block_c = block_sum(mine_c, sh);
  unsigned long long* ac_counts = p.block_counts + 1 * kMaxFinalizeBlocks;
  if (threadIdx.x == 0) ac_counts[blk] = (block_a << 32) | block_c;
  if (!grid_barrier(p.ctl, ++barriers * G, sh)) return;

  // ---------------- phase 5: write the survivors in index order ----------------
  unsigned long long a_before = 0, c_before = 0, a_all = 0, c_all = 0;
  for (unsigned int b = threadIdx.x; b < G; b += kCta) {
    const unsigned long long w = ld_cg_u64(ac_counts + b);
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
  const unsigned int lt = (1u << lane) - 1u;
  for (unsigned int seg = s0 + warp; seg < s1; seg += kCta / 32) {
    unsigned long long a_done = a_before, c_done = c_before;
    for (unsigned int s = 0; s < seg - s0; ++s) {
      a_done += sh.seg_a[s];
      c_done += sh.seg_c[s];
    }
    const unsigned int cnt = __ldcg(p.seg_count + seg);
    const unsigned long long base = warp_first_round(seg, p.segments, rounds) * kRound;
    for (unsigned int i0 = 0; i0 < cnt; i0 += 32) {
      const unsigned int i = i0 + lane;
      uint32_t bits = 0, key = 0;
      if (i < cnt) {
        bits = __ldcg(p.seg_val + base + i);
        key = bits & 0x7FFFFFFFu;
      }
      const bool a = i < cnt && key > T;
      const bool c = i < cnt && key == T;
      const unsigned int ba = __ballot_sync(0xFFFFFFFFu, a);
      const unsigned int bc = __ballot_sync(0xFFFFFFFFu, c);
      const unsigned long long a_here = a_done + __popc(ba & lt);
      const unsigned long long c_here = c_done + __popc(bc & lt);
      if (a || (c && c_here < r)) {
        const unsigned long long pos = a_here + min(c_here, r);
        out_idx[pos] = __ldcg(p.seg_idx + base + i);
        p.raw_val[pos] = __uint_as_float(bits);
      }
      a_done += __popc(ba);
      c_done += __popc(bc);
    }
  }
  if (!grid_barrier(p.ctl, ++barriers * G, sh)) return;

  // ---------------- phase 6: quantise, write the header ----------------
  if (blk == 0 && threadIdx.x == 0) {
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
  const unsigned long long qblocks = (p.k + NSML_QBLOCK - 1) / NSML_QBLOCK;
  for (unsigned long long qb = blk; qb < qblocks; qb += G) {
    const unsigned long long j0 = qb * NSML_QBLOCK + threadIdx.x * 4;
    float v[4] = {0.f, 0.f, 0.f, 0.f};
    int cnt = 0;
    if (j0 + 4 <= p.k) {
      const float4 f = __ldcg(reinterpret_cast<const float4*>(p.raw_val + j0));
      v[0] = f.x; v[1] = f.y; v[2] = f.z; v[3] = f.w;
      cnt = 4;
    } else if (j0 < p.k) {
      cnt = (int)(p.k - j0);
      for (int e = 0; e < cnt; ++e) v[e] = __ldcg(p.raw_val + j0 + e);
    }
    if (p.bits == NSML_BITS_FP16) {
      uint16_t* out = reinterpret_cast<uint16_t*>(p.payload + p.P.val_off);
      if (cnt == 4) {
        uint2 w;
        w.x = (uint32_t)encode_f16(v[0]) | ((uint32_t)encode_f16(v[1]) << 16);
        w.y = (uint32_t)encode_f16(v[2]) | ((uint32_t)encode_f16(v[3]) << 16);
        *reinterpret_cast<uint2*>(out + j0) = w;
      } else {
        for (int e = 0; e < cnt; ++e) out[j0 + e] = encode_f16(v[e]);
      }
      continue;
    }
    // block max-abs: warp shuffles, then one value per warp through shared memory
    float m = fmaxf(fmaxf(fabsf(v[0]), fabsf(v[1])), fmaxf(fabsf(v[2]), fabsf(v[3])));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
    __syncthreads();  // qmax of the previous block of survivors has been read
    if (lane == 0) sh.qmax[warp] = m;
    __syncthreads();
    m = sh.qmax[0];
#pragma unroll
    for (int w = 1; w < kCta / 32; ++w) m = fmaxf(m, sh.qmax[w]);
    const float scale = __fdiv_rn(m, 127.0f);
    if (threadIdx.x == 0) reinterpret_cast<float*>(p.payload + p.P.scale_off)[qb] = scale;
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

}  // namespace nsml
