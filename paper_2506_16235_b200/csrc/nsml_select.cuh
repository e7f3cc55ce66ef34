// Radix-select threshold search on the magnitude keys (Alg. 2 Step 3: which
// k = ceil(ratio*n) gradients have the largest absolute value).
//
// Level 0 histograms the top digit over the whole bucket; the block that
// finishes last resolves the bin that holds the k-th largest key.  The bucket
// compaction then keeps every key in or above that bin (a superset of the
// survivors); levels 1 and 2 histogram the remaining digits over that short
// list only, which pins the exact threshold key T and the tie budget r.
#pragma once

#include "nsml_common.cuh"

namespace nsml {

// Called by all threads of the last block of a histogram level.  Finds the
// digit d with  #{digit > d} < k_rem <= #{digit >= d}  among the keys that
// match the current prefix, and advances the selection state.
template <int LEVEL>
__device__ void resolve_level(Ctl* ctl, const unsigned int* ghist, unsigned long long k_first) {
  constexpr int NB = 1 << digit_bits(LEVEL);
  constexpr int PER = (NB + kCta - 1) / kCta;
  __shared__ unsigned long long s_part[kCta];
  const int t = threadIdx.x;

  unsigned long long part = 0;
#pragma unroll
  for (int b = 0; b < PER; ++b) {
    int bin = t * PER + b;
    if (bin < NB) part += __ldcg(ghist + bin);
  }
  s_part[t] = part;
  __syncthreads();

  if (t == 0) {
    const unsigned long long k_rem = (LEVEL == 0) ? k_first : ctl->k_rem;
    unsigned long long above = 0;
    int chunk = kCta - 1;
    for (; chunk > 0; --chunk) {
      if (above + s_part[chunk] >= k_rem) break;
      above += s_part[chunk];
    }
    int d = min(NB - 1, chunk * PER + PER - 1);
    for (; d > chunk * PER; --d) {
      unsigned long long c = __ldcg(ghist + d);
      if (above + c >= k_rem) break;
      above += c;
    }
    // `above` keys are strictly above digit d; the k_rem-th largest is in d.
    const unsigned long long in_bin = __ldcg(ghist + d);
    unsigned long long rem = k_rem - above;  // 1 <= rem <= in_bin
    const unsigned int prefix = (LEVEL == 0) ? (unsigned)d : ((ctl->prefix << digit_bits(LEVEL)) | (unsigned)d);
    ctl->prefix = prefix;

    if (LEVEL == 0) {
      unsigned int lo = prefix << digit_shift(0);
      const unsigned int hi = (prefix + 1u) << digit_shift(0);
      unsigned long long r = ~0ull;  // keep every key of the boundary bin
      unsigned int exact = 0;
      if (d == 0) {
        // The boundary bin holds the zeros.  If the non-zero keys run out
        // before k is reached the threshold key is exactly 0 and the tie
        // budget is known now; otherwise zeros are certainly not survivors.
        const unsigned long long nz = in_bin - *(volatile unsigned long long*)&ctl->zero_count;
        if (rem > nz) {
          lo = 0;
          r = rem - nz;
          exact = 1;
          ctl->lo = 0;
          ctl->hi = 1;
          rem = r;
        } else {
          lo = 1;
        }
      }
      if (!exact) {
        ctl->lo = lo;
        ctl->hi = hi;
      }
      ctl->r = r;
      ctl->exact = exact;
      ctl->k_rem = rem;
    } else if (LEVEL == 1) {
      ctl->k_rem = rem;
    } else {
      // all 31 bits resolved: T = prefix, take the first `rem` ties by index
      ctl->k_rem = rem;
      ctl->lo = prefix;
      ctl->hi = prefix + 1u;
      ctl->r = rem;
      ctl->exact = 1;
    }
  }
}

// Histogram of digit LEVEL over the elements of `src` whose higher digits equal
// the resolved prefix.  LEVEL 0 runs over the bucket and also counts zero keys
// and flags non-finite input; LEVEL 1 and 2 run over the candidate list.
template <int LEVEL, class Src>
__global__ void __launch_bounds__(kCta)
k_histogram(Src src, unsigned long long count_arg, unsigned long long k, Ctl* ctl, unsigned int* ghist_all) {
  constexpr int NB = 1 << digit_bits(LEVEL);
  constexpr int SHIFT = digit_shift(LEVEL);
  __shared__ unsigned int s_hist[NB];
  __shared__ bool s_last;

  unsigned int* ghist = ghist_all + LEVEL * kMaxBins;
  unsigned long long count = count_arg;
  unsigned int want_prefix = 0;
  if (LEVEL > 0) {
    if (ctl->exact) return;  // threshold already final
    count = ctl->list_count;
    want_prefix = ctl->prefix;
  }

  for (int b = threadIdx.x; b < NB; b += kCta) s_hist[b] = 0;
  __syncthreads();

  unsigned int zeros = 0;
  bool nonfinite = false;
  const unsigned long long stride = (unsigned long long)gridDim.x * kCta * 4;
  for (unsigned long long i0 = ((unsigned long long)blockIdx.x * kCta + threadIdx.x) * 4; i0 < count; i0 += stride) {
    Quad q = src.load4(i0, count);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      if (!(q.valid & (1u << e))) continue;
      const uint32_t key = q.bits[e] & 0x7FFFFFFFu;
      if (LEVEL == 0) {
        zeros += (key == 0);
        nonfinite |= (key >= kInfKey);
        atomicAdd(&s_hist[key >> SHIFT], 1u);
      } else {
        if ((key >> (SHIFT + digit_bits(LEVEL))) == want_prefix)
          atomicAdd(&s_hist[(key >> SHIFT) & (NB - 1)], 1u);
      }
    }
  }
  if (LEVEL == 0) {
    for (int o = 16; o > 0; o >>= 1) zeros += __shfl_down_sync(0xFFFFFFFFu, zeros, o);
    if ((threadIdx.x & 31) == 0 && zeros) atomicAdd(&ctl->zero_count, (unsigned long long)zeros);
    if (nonfinite) set_status(&ctl->status, NSML_ERR_NONFINITE);
  }
  __syncthreads();
  for (int b = threadIdx.x; b < NB; b += kCta) {
    unsigned int c = s_hist[b];
    if (c) atomicAdd(&ghist[b], c);
  }

  // the block that arrives last sees every block's contribution
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) s_last = (atomicAdd(&ctl->done[LEVEL], 1u) == gridDim.x - 1);
  __syncthreads();
  if (s_last) {
    __threadfence();
    resolve_level<LEVEL>(ctl, ghist, k);
  }
}

}  // namespace nsml
