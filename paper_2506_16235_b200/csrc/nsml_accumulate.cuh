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

struct PayloadTable {
  const unsigned char* p[NSML_MAX_WORKERS];
  unsigned long long bytes[NSML_MAX_WORKERS];  // size of the buffer behind p[w]; 0 = not known
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

// A header is accepted when its fields describe a payload for this n in the layout nsml_compress writes
// and, where the size of the buffer is known (bytes != 0), that layout fits the buffer: a truncated
// payload, or one whose k field was corrupted upwards, is then refused before anything behind the header
// is read.
__host__ __device__ inline bool header_ok(const nsml_payload_header* h, unsigned long long n, unsigned long long bytes = 0) {
  if (h->magic != NSML_PAYLOAD_MAGIC || h->version != NSML_PAYLOAD_VERSION) return false;
  if (h->n != n || h->k < 1 || h->k > n || h->qblock != NSML_QBLOCK) return false;
  if (h->bits != NSML_BITS_INT8 && h->bits != NSML_BITS_FP16 && h->bits != NSML_BITS_FP32) return false;
  const unsigned long long k = h->k;
  const unsigned long long val_off = 64 + (k * 4 + 15) / 16 * 16;
  if (h->idx_off != 64 || h->val_off != val_off) return false;
  unsigned long long total;
  if (h->bits == NSML_BITS_INT8) {
    const unsigned long long nblocks = (k + NSML_QBLOCK - 1) / NSML_QBLOCK;
    if (h->nblocks != nblocks) return false;
    if (h->scale_off != val_off + (k + 15) / 16 * 16) return false;
    total = h->scale_off + (nblocks * 4 + 15) / 16 * 16;
  } else {
    total = val_off + (k * (h->bits == NSML_BITS_FP32 ? 4 : 2) + 15) / 16 * 16;
  }
  return bytes == 0 || total <= bytes;
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
  if (!header_ok(h, n, table.bytes[w])) {
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
  if (!header_ok(h, n, table.bytes[w])) {
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

// What a block needs to know about one worker's payload, read from its header once per block.
struct WorkerView {
  const uint32_t* idx;
  const unsigned char* val;  // int8 codes, binary16 bit patterns or float32 values
  const float* scale;
  int bits;
};

constexpr int kMergeUnits = 8;  // (worker, 256-entry chunk) units a thread loads before the adds are applied

__global__ void __launch_bounds__(kCta, 6)
k_merge(PayloadTable table, int W, float* __restrict__ dense, unsigned long long n, int zero_first,
        unsigned int tiles, const unsigned int* __restrict__ offsets, int* status) {
  __shared__ __align__(16) float s_acc[kDenseTile];
  __shared__ WorkerView s_view[NSML_MAX_WORKERS];
  __shared__ unsigned int s_from[NSML_MAX_WORKERS], s_to[NSML_MAX_WORKERS], s_pref[NSML_MAX_WORKERS + 1];
  const unsigned long long per = (unsigned long long)tiles + 1;
  bool bad = false;
  if (threadIdx.x < W) {
    // Headers are checked here (the partition kernel cleared the status word).  A worker with a bad
    // header has all-zero offsets, so its view is never used.
    const unsigned char* pbase = table.p[threadIdx.x];
    const nsml_payload_header* h = reinterpret_cast<const nsml_payload_header*>(pbase);
    WorkerView v = {nullptr, nullptr, nullptr, 0};
    if (header_ok(h, n, table.bytes[threadIdx.x])) {
      v.idx = reinterpret_cast<const uint32_t*>(pbase + h->idx_off);
      v.val = pbase + h->val_off;
      v.scale = reinterpret_cast<const float*>(pbase + h->scale_off);
      v.bits = (int)h->bits;
    } else {
      bad = blockIdx.x == 0;
    }
    s_view[threadIdx.x] = v;
  }

  // offsets of the block's next tile, fetched by the first warp one tile ahead (two workers per lane), so that a
  // tile costs one round trip to memory (its entries) instead of two
  unsigned int ahead_a[2] = {0, 0}, ahead_b[2] = {0, 0};
  if (threadIdx.x < 32 && blockIdx.x < tiles) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int w = threadIdx.x * 2 + h;
      if (w < W) {
        ahead_a[h] = offsets[w * per + blockIdx.x];
        ahead_b[h] = offsets[w * per + blockIdx.x + 1];
      }
    }
  }
  for (unsigned int tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
    const unsigned long long lo = (unsigned long long)tile * kDenseTile;
    const unsigned int len = (unsigned int)min((unsigned long long)kDenseTile, n - lo);
    __syncthreads();  // the previous tile is fully written out (first tile: the views are in place)
    if (threadIdx.x < 32) {
      // the first warp hands out the tile's offsets and scans the counts
      unsigned int cnt[2];
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int w = threadIdx.x * 2 + h;
        cnt[h] = 0;
        if (w < W) {
          unsigned int a = ahead_a[h];
          unsigned int b = ahead_b[h];
          const unsigned long long next = (unsigned long long)tile + gridDim.x;
          if (next < tiles) {
            ahead_a[h] = offsets[w * per + next];
            ahead_b[h] = offsets[w * per + next + 1];
          }
          if (b < a) b = a;  // only a corrupt (unsorted) payload gets here
          s_from[w] = a;
          s_to[w] = b;
          cnt[h] = b - a;
        }
      }
      unsigned int incl = cnt[0] + cnt[1];
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const unsigned int up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if ((int)threadIdx.x >= o) incl += up;
      }
      const unsigned int before = incl - cnt[0] - cnt[1];
      if ((int)threadIdx.x * 2 < W) s_pref[threadIdx.x * 2] = before;
      if ((int)threadIdx.x * 2 + 1 < W) s_pref[threadIdx.x * 2 + 1] = before + cnt[0];
      static_assert(NSML_MAX_WORKERS == 64, "two workers per lane of the first warp");
      if (threadIdx.x == 31) s_pref[W] = incl;
    }
    __syncthreads();
    const unsigned int total = s_pref[W];
    if (total == 0 && !zero_first) continue;
    // Few entries: touch only their elements in global memory (after zero-filling
    // the tile there in overwrite mode).  Many entries: stage the tile in
    // shared memory and write it back in one sweep.
    const bool staged = (unsigned long long)total * 64 > len;
    float* dtile = dense + lo;
    if (staged) {
      for (unsigned int i = threadIdx.x * 4; i < len; i += kCta * 4) {
        if (i + 4 <= len) {
          float4 v = zero_first ? make_float4(0.f, 0.f, 0.f, 0.f) : *reinterpret_cast<const float4*>(dtile + i);
          *reinterpret_cast<float4*>(s_acc + i) = v;
        } else {
          for (unsigned int e = i; e < len; ++e) s_acc[e] = zero_first ? 0.f : dtile[e];
        }
      }
    } else if (zero_first) {
      for (unsigned int i = threadIdx.x * 4; i < len; i += kCta * 4) {
        if (i + 4 <= len) *reinterpret_cast<float4*>(dtile + i) = make_float4(0.f, 0.f, 0.f, 0.f);
        else for (unsigned int e = i; e < len; ++e) dtile[e] = 0.f;
      }
    }
    __syncthreads();  // the tile's starting values are in place before any add reads them

    // The tile's entries are taken worker by worker in units of kCta consecutive entries, one per
    // thread.  A thread first issues the loads of its entries of the next kMergeUnits units and
    // touches none of the results, so that a group of units costs one memory latency; then the adds
    // are applied unit by unit with a block barrier wherever the worker changes: an element gets at
    // most one add per worker, always in worker order.
    float* acc = staged ? s_acc : dtile;
    int w = 0;           // current worker (uniform over the block)
    unsigned int c = 0;  // entries of worker w already taken
    while (w < W && s_to[w] == s_from[w]) ++w;
    while (w < W) {
      uint32_t raw_idx[kMergeUnits];  // 0xFFFFFFFF = no entry (indices are below 2^31)
      int raw_val[kMergeUnits];
      float raw_scale[kMergeUnits];
      int unit_w[kMergeUnits], unit_bits[kMergeUnits];
#pragma unroll
      for (int u = 0; u < kMergeUnits; ++u) {
        unit_w[u] = w;
        unit_bits[u] = 0;
        raw_idx[u] = 0xFFFFFFFFu;
        raw_val[u] = 0;
        raw_scale[u] = 0.f;
        if (w < W) {
          const unsigned int to = s_to[w];
          const unsigned int j = s_from[w] + c + threadIdx.x;
          const WorkerView v = s_view[w];
          unit_bits[u] = v.bits;
          if (j < to) {
            raw_idx[u] = v.idx[j];
            if (v.bits == NSML_BITS_INT8) {
              raw_val[u] = reinterpret_cast<const signed char*>(v.val)[j];
              raw_scale[u] = v.scale[j >> 10];
            } else if (v.bits == NSML_BITS_FP16) {
              raw_val[u] = reinterpret_cast<const uint16_t*>(v.val)[j];
            } else {
              raw_val[u] = reinterpret_cast<const int*>(v.val)[j];  // float32 bit pattern
            }
          }
          c += kCta;
          if (s_from[w] + c >= to) {  // worker w is used up: on to the next one that has entries here
            c = 0;
            do ++w; while (w < W && s_to[w] == s_from[w]);
          }
        }
      }
#pragma unroll
      for (int u = 0; u < kMergeUnits; ++u) {
        if (unit_w[u] >= W) break;
        if (raw_idx[u] != 0xFFFFFFFFu) {
          const unsigned long long o = (unsigned long long)raw_idx[u] - lo;  // wraps if idx < lo
          const float v = unit_bits[u] == NSML_BITS_INT8   ? decode_i8(raw_val[u], raw_scale[u])
                          : unit_bits[u] == NSML_BITS_FP16 ? decode_f16((uint16_t)raw_val[u])
                                                           : __int_as_float(raw_val[u]);
          if (o < len) acc[o] += v; else bad = true;
        }
        if (u + 1 == kMergeUnits || unit_w[u + 1] != unit_w[u]) __syncthreads();  // uniform over the block
      }
    }

    if (staged) {
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
