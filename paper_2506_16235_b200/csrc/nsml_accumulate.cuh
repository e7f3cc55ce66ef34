// Decompress and sum the W gathered payloads into one dense float32 gradient
// (Section 4.2 Step 3 "further aggregation"; with top-k payloads every worker
// receives all payloads, the AllGather pattern of Section 5.3, and sums them).
//
// Payload indices are ascending, so the work is split by dense range instead
// of by payload entry: a block owns a tile of the dense buffer, finds each
// worker's entries for that tile from a precomputed offset table, adds them in
// worker order in shared memory and writes the tile once, coalesced.  No
// atomics, fixed summation order, and in overwrite mode the zero fill costs
// nothing extra.
#pragma once

#include "nsml_common.cuh"
#include "nsml_codec.cuh"

namespace nsml {

constexpr int kDenseTile = 8192;  // dense elements per block iteration (32 KB of shared memory)
constexpr int kMergeRound = 4 * kCta;  // payload entries a block loads before applying them

struct PayloadTable {
  const unsigned char* p[NSML_MAX_WORKERS];
};

struct AccumulateLayout {
  size_t offsets;  // u32[W][tiles + 1]
  size_t total;
};

inline AccumulateLayout accumulate_layout(int64_t n, int W) {
  AccumulateLayout L;
  size_t tiles = (size_t)((n + kDenseTile - 1) / kDenseTile);
  L.offsets = 256;
  L.total = L.offsets + align_up((size_t)W * (tiles + 1) * 4, 256);
  return L;
}

__device__ inline bool header_ok(const nsml_payload_header* h, unsigned long long n) {
  if (h->magic != NSML_PAYLOAD_MAGIC || h->version != NSML_PAYLOAD_VERSION) return false;
  if (h->n != n || h->k < 1 || h->k > n || h->qblock != NSML_QBLOCK) return false;
  if (h->bits != NSML_BITS_INT8 && h->bits != NSML_BITS_FP16) return false;
  const unsigned long long k = h->k;
  const unsigned long long val_off = 64 + (k * 4 + 15) / 16 * 16;
  if (h->idx_off != 64 || h->val_off != val_off) return false;
  if (h->bits == NSML_BITS_INT8) {
    if (h->nblocks != (k + NSML_QBLOCK - 1) / NSML_QBLOCK) return false;
    if (h->scale_off != val_off + (k + 15) / 16 * 16) return false;
  }
  return true;
}

// offsets[w][b] = first payload entry of worker w whose index is >= b*kDenseTile.
// The partition kernels also clear the call's status word (no separate clearing
// step is needed); payload errors are therefore reported by the merge kernel,
// which starts only after every block here has finished: a worker with a bad
// header gets all-zero offsets, so nothing of its payload is read.
// One warp per (worker, boundary): a 33-way search, every lane probing one
// position per step, so a boundary costs about log33(k) memory round trips
// instead of log2(k).
__global__ void __launch_bounds__(kCta)
k_partition(PayloadTable table, int W, unsigned long long n, unsigned int tiles, unsigned int* offsets, int* status) {
  const int lane = threadIdx.x & 31;
  if (blockIdx.x == 0 && threadIdx.x == 0) *status = NSML_OK;
  const unsigned long long g = ((unsigned long long)blockIdx.x * kCta + threadIdx.x) >> 5;  // one warp per offset
  const unsigned long long per = (unsigned long long)tiles + 1;
  if (g >= per * W) return;  // whole warps leave together
  const int w = (int)(g / per);
  const unsigned long long b = g % per;
  const nsml_payload_header* h = reinterpret_cast<const nsml_payload_header*>(table.p[w]);
  if (!header_ok(h, n)) {
    if (lane == 0) offsets[g] = 0;
    return;
  }
  const uint32_t* idx = reinterpret_cast<const uint32_t*>(table.p[w] + h->idx_off);
  const unsigned long long target = b * kDenseTile;
  unsigned long long lo = 0, hi = h->k;  // the answer lies in [lo, hi]
  while (hi - lo > 32) {
    const unsigned long long width = hi - lo;
    const unsigned long long probe = lo + (lane + 1) * width / 33;  // lo < probe < hi, ascending with the lane
    const unsigned int below = __ballot_sync(0xFFFFFFFFu, idx[probe] < target);
    const int c = __popc(below);  // ascending indices: the lanes below the target form a prefix
    const unsigned long long new_lo = (c == 0) ? lo : lo + (unsigned long long)c * width / 33 + 1;
    const unsigned long long new_hi = (c == 32) ? hi : lo + (unsigned long long)(c + 1) * width / 33;
    lo = new_lo;
    hi = new_hi;
  }
  const bool below = (lo + lane < hi) && idx[lo + lane] < target;
  const unsigned int rest = __ballot_sync(0xFFFFFFFFu, below);
  if (lane == 0) offsets[g] = (unsigned int)(lo + __popc(rest));
}

// The same table with one thread per offset and a plain binary search: less
// latency-efficient per offset, but with hundreds of thousands of offsets the
// searches hide each other's latency and 32 times fewer threads are needed.
__global__ void __launch_bounds__(kCta)
k_partition_wide(PayloadTable table, int W, unsigned long long n, unsigned int tiles, unsigned int* offsets, int* status) {
  if (blockIdx.x == 0 && threadIdx.x == 0) *status = NSML_OK;
  const unsigned long long g = (unsigned long long)blockIdx.x * kCta + threadIdx.x;
  const unsigned long long per = (unsigned long long)tiles + 1;
  if (g >= per * W) return;
  const int w = (int)(g / per);
  const unsigned long long b = g % per;
  const nsml_payload_header* h = reinterpret_cast<const nsml_payload_header*>(table.p[w]);
  if (!header_ok(h, n)) {
    offsets[g] = 0;
    return;
  }
  const uint32_t* idx = reinterpret_cast<const uint32_t*>(table.p[w] + h->idx_off);
  const unsigned long long target = b * kDenseTile;
  unsigned long long lo = 0, hi = h->k;
  while (lo < hi) {
    const unsigned long long mid = (lo + hi) >> 1;
    if (idx[mid] < target) lo = mid + 1; else hi = mid;
  }
  offsets[g] = (unsigned int)lo;
}

__global__ void __launch_bounds__(kCta)
k_merge(PayloadTable table, int W, float* __restrict__ dense, unsigned long long n, int zero_first,
        unsigned int tiles, const unsigned int* __restrict__ offsets, int* status) {
  __shared__ __align__(16) float s_acc[kDenseTile];
  __shared__ unsigned int s_from[NSML_MAX_WORKERS], s_to[NSML_MAX_WORKERS];
  __shared__ unsigned int s_total;
  const unsigned long long per = (unsigned long long)tiles + 1;
  bool bad = false;
  if (blockIdx.x == 0 && threadIdx.x < W)  // headers are checked here; the partition kernel cleared the status
    bad = !header_ok(reinterpret_cast<const nsml_payload_header*>(table.p[threadIdx.x]), n);

  for (unsigned int tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
    const unsigned long long lo = (unsigned long long)tile * kDenseTile;
    const unsigned int len = (unsigned int)min((unsigned long long)kDenseTile, n - lo);
    __syncthreads();  // the previous tile is fully written out
    if (threadIdx.x == 0) s_total = 0;
    __syncthreads();
    if (threadIdx.x < W) {
      unsigned int a = offsets[threadIdx.x * per + tile];
      unsigned int b = offsets[threadIdx.x * per + tile + 1];
      if (b < a) b = a;  // only a corrupt (unsorted) payload gets here
      s_from[threadIdx.x] = a;
      s_to[threadIdx.x] = b;
      if (b > a) atomicAdd(&s_total, b - a);
    }
    __syncthreads();
    const unsigned int total = s_total;
    if (total == 0 && !zero_first) continue;
    // Few entries: touch only their elements in global memory (after zero-filling
    // the tile there in overwrite mode).  Many entries: stage the whole tile in
    // shared memory and write it back in one sweep.
    const bool staged = (unsigned long long)total * 16 > len;
    if (!staged && zero_first) {
      float* dtile = dense + lo;
      for (unsigned int i = threadIdx.x * 4; i < len; i += kCta * 4) {
        if (i + 4 <= len) *reinterpret_cast<float4*>(dtile + i) = make_float4(0.f, 0.f, 0.f, 0.f);
        else for (unsigned int e = i; e < len; ++e) dtile[e] = 0.f;
      }
      __syncthreads();  // the zeros are in place before any add reads them
    }

    if (staged) {
      float* dtile = dense + lo;
      for (unsigned int i = threadIdx.x * 4; i < len; i += kCta * 4) {
        if (i + 4 <= len) {
          float4 v = zero_first ? make_float4(0.f, 0.f, 0.f, 0.f) : *reinterpret_cast<const float4*>(dtile + i);
          *reinterpret_cast<float4*>(s_acc + i) = v;
        } else {
          for (unsigned int e = i; e < len; ++e) s_acc[e] = zero_first ? 0.f : dtile[e];
        }
      }
      __syncthreads();
    }

    // The tile's entries of all workers, taken as one worker-major sequence of
    // `total` entries, are processed kMergeRound at a time: every thread first
    // loads its (up to 4) entries, so that one round costs one memory latency,
    // then the adds are applied worker by worker (an element may receive one
    // add per worker; within a worker indices are distinct).
    for (unsigned int base = 0; base < total; base += kMergeRound) {
      unsigned int off[4];
      float val[4];
      int wk[4];
      int w_min = W, w_max = -1;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const unsigned int f = base + e * kCta + threadIdx.x;  // position in the flattened sequence
        wk[e] = -1;
        if (f < total) {
          int w = 0;
          unsigned int before = 0;
          while (before + (s_to[w] - s_from[w]) <= f) { before += s_to[w] - s_from[w]; ++w; }  // w < W because f < total
          const unsigned int j = s_from[w] + (f - before);
          const unsigned char* pbase = table.p[w];
          const nsml_payload_header* h = reinterpret_cast<const nsml_payload_header*>(pbase);
          const unsigned long long o = (unsigned long long)reinterpret_cast<const uint32_t*>(pbase + h->idx_off)[j] - lo;  // wraps if idx < lo
          float v;
          if (h->bits == NSML_BITS_INT8)
            v = decode_i8(reinterpret_cast<const signed char*>(pbase + h->val_off)[j],
                          reinterpret_cast<const float*>(pbase + h->scale_off)[j >> 10]);
          else
            v = decode_f16(reinterpret_cast<const uint16_t*>(pbase + h->val_off)[j]);
          if (o < len) {
            wk[e] = w;
            off[e] = (unsigned int)o;
            val[e] = v;
          } else {
            bad = true;
          }
        }
      }
      // workers present in this round (the sequence is worker-major, so they form a range)
      {
        const unsigned int f_lo = base, f_hi = min(total, base + kMergeRound) - 1;
        unsigned int before = 0;
        for (int w = 0; w < W; ++w) {
          const unsigned int c = s_to[w] - s_from[w];
          if (c && before <= f_hi && before + c > f_lo) { w_min = min(w_min, w); w_max = max(w_max, w); }
          before += c;
        }
      }
      for (int w = w_min; w <= w_max; ++w) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          if (wk[e] == w) {
            if (staged) s_acc[off[e]] += val[e]; else dense[lo + off[e]] += val[e];
          }
        }
        __syncthreads();  // worker w is done before worker w+1 adds to the same elements
      }
    }

    if (staged) {
      float* dtile = dense + lo;
      for (unsigned int i = threadIdx.x * 4; i < len; i += kCta * 4) {
        if (i + 4 <= len) {
          *reinterpret_cast<float4*>(dtile + i) = *reinterpret_cast<const float4*>(s_acc + i);
        } else {
          for (unsigned int e = i; e < len; ++e) dtile[e] = s_acc[e];
        }
      }
    }
  }
  if (bad) set_status(status, NSML_ERR_PAYLOAD);
}

}  // namespace nsml
