// libnsml C ABI: argument checks, workspace carving and kernel launches.
// See include/nsml.h for the contract of every entry point.
#include <atomic>
#include <cmath>
#include <cstring>
#include <mutex>
#include <vector>

#include "nsml_accumulate.cuh"
#include "nsml_adaptive.cuh"
#include "nsml_codec.cuh"
#include "nsml_common.cuh"
#include "nsml_compact.cuh"
#include "nsml_finalize.cuh"
#include "nsml_dense.cuh"
#include "nsml_select.cuh"

namespace nsml {

enum KernelId {
  K_SAMPLE = 0, K_COMPACT_BUCKET, K_FINALIZE, K_PARTITION, K_MERGE, K_CLEAR, K_FINALIZE_DENSE,
  K_SUMSQ, K_FEEDBACK_ADD, K_FEEDBACK_SUBTRACT, K_PRUNE_HIST, K_PRUNE_TIES, K_PRUNE_WRITE, K_PRUNE_WRITE_RANKED, K_GATHER, K_PRUNE_SAMPLE, K_PRUNE_COUNT, K_PRUNE_SETTLE, K_PRUNE_MARK, K_PRUNE_FIX, K_COUNT
};

static const char* const kKernelNames[K_COUNT] = {"k_sample", "k_compact_bucket", "k_finalize", "k_partition", "k_merge",
                                                  "k_clear", "k_finalize_dense", "k_sumsq", "k_feedback_add",
                                                  "k_feedback_subtract", "k_prune_hist", "k_prune_ties", "k_prune_write",
                                                  "k_prune_write_ranked", "k_gather", "k_prune_sample", "k_prune_count",
                                                  "k_prune_settle", "k_prune_mark", "k_prune_fix"};

static std::atomic<int64_t> g_launches{0};

// ---- optional per-kernel timing with CUDA events --------------------------
struct ProfRecord {
  int id;
  cudaEvent_t start, stop;
};
static std::mutex g_prof_mutex;
static std::atomic<bool> g_prof_on{false};
static std::vector<ProfRecord> g_prof_records;
static double g_prof_ms[K_COUNT];
static int64_t g_prof_launches[K_COUNT];

static void prof_drain_locked() {
  for (ProfRecord& r : g_prof_records) {
    float ms = 0.f;
    if (cudaEventSynchronize(r.stop) == cudaSuccess && cudaEventElapsedTime(&ms, r.start, r.stop) == cudaSuccess) {
      g_prof_ms[r.id] += ms;
      g_prof_launches[r.id] += 1;
    }
    cudaEventDestroy(r.start);
    cudaEventDestroy(r.stop);
  }
  g_prof_records.clear();
}

struct LaunchScope {  // brackets one kernel launch
  int id;
  cudaStream_t stream;
  cudaEvent_t start = nullptr, stop = nullptr;
  // timed = false: never bracket this launch with events (creating events allocates)
  LaunchScope(int id_, cudaStream_t s, bool timed = true) : id(id_), stream(s) {
    if (timed && g_prof_on.load(std::memory_order_relaxed)) {
      cudaEventCreate(&start);
      cudaEventCreate(&stop);
      cudaEventRecord(start, stream);
    }
  }
  ~LaunchScope() {
    g_launches.fetch_add(1, std::memory_order_relaxed);
    if (start) {
      cudaEventRecord(stop, stream);
      std::lock_guard<std::mutex> lock(g_prof_mutex);
      g_prof_records.push_back({id, start, stop});
    }
  }
};

// ---- per-device launch geometry -------------------------------------------
struct DeviceInfo {
  bool ready = false;
  int sms = 0;
  int compact_feedback = 0, finalize_small = 0, finalize_large = 0, merge = 0;  // resident blocks per SM
  int sumsq = 0, feedback_add = 0, prune_hist = 0, prune_write = 0, prune_write_ranked = 0;  // the same, streaming kernels
  bool finalize_cluster = false;  // the one-cluster shape of the list stage fits an SM
};
static DeviceInfo g_dev[64];
static std::mutex g_dev_mutex;

static int device_info(const DeviceInfo** out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return NSML_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_dev_mutex);
  DeviceInfo& d = g_dev[dev];
  if (!d.ready) {
    if (cudaDeviceGetAttribute(&d.sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return NSML_ERR_CUDA;
    cudaError_t e = cudaSuccess;
    e = cudaFuncSetAttribute(k_compact_bucket<NSML_F32, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kCompactFeedbackSmem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_compact_bucket<NSML_BF16, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kCompactFeedbackSmem);
    if (e == cudaSuccess) e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&d.compact_feedback, k_compact_bucket<NSML_F32, true>, kCta, kCompactFeedbackSmem);
    auto prepare = [&](auto kernel, int threads, int cache, int* resident) {
      if (e == cudaSuccess) e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)finalize_dyn_smem(cache));
      int r = 0;
      if (e == cudaSuccess) e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&r, kernel, threads, finalize_dyn_smem(cache));
      if (*resident == 0 || r < *resident) *resident = r;
    };
    prepare(k_finalize<NSML_F32, kFinSmallThreads, kFinSmallCache>, kFinSmallThreads, kFinSmallCache, &d.finalize_small);
    prepare(k_finalize<NSML_BF16, kFinSmallThreads, kFinSmallCache>, kFinSmallThreads, kFinSmallCache, &d.finalize_small);
    prepare(k_finalize_dense<NSML_F32, kFinSmallThreads, kFinSmallCache>, kFinSmallThreads, kFinSmallCache, &d.finalize_small);
    prepare(k_finalize_dense<NSML_BF16, kFinSmallThreads, kFinSmallCache>, kFinSmallThreads, kFinSmallCache, &d.finalize_small);
    int cluster_shape = 0;
    prepare(k_finalize<NSML_F32, kFinClusterThreads, kFinClusterCache, true>, kFinClusterThreads, kFinClusterCache, &cluster_shape);
    prepare(k_finalize<NSML_BF16, kFinClusterThreads, kFinClusterCache, true>, kFinClusterThreads, kFinClusterCache, &cluster_shape);
    d.finalize_cluster = cluster_shape >= 1;
    prepare(k_finalize<NSML_F32, kFinLargeThreads, kFinLargeCache>, kFinLargeThreads, kFinLargeCache, &d.finalize_large);
    prepare(k_finalize<NSML_BF16, kFinLargeThreads, kFinLargeCache>, kFinLargeThreads, kFinLargeCache, &d.finalize_large);
    prepare(k_finalize_dense<NSML_F32, kFinLargeThreads, kFinDenseLargeCache>, kFinLargeThreads, kFinDenseLargeCache, &d.finalize_large);
    prepare(k_finalize_dense<NSML_BF16, kFinLargeThreads, kFinDenseLargeCache>, kFinLargeThreads, kFinDenseLargeCache, &d.finalize_large);
    if (e == cudaSuccess) e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&d.merge, k_merge, kCta, 0);
    // The streaming kernels run as one wave of resident blocks (a second, partial wave would read
    // with a fraction of the SMs' loads in flight).
    auto resident = [&](auto kernel, int* out) {
      int r = 0;
      if (e == cudaSuccess) e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&r, kernel, kCta, 0);
      if (*out == 0 || r < *out) *out = r;
    };
    resident(k_sumsq<NSML_F32>, &d.sumsq);
    resident(k_sumsq<NSML_BF16>, &d.sumsq);
    resident(k_feedback_add<NSML_F32>, &d.feedback_add);
    resident(k_feedback_add<NSML_BF16>, &d.feedback_add);
    resident(k_prune_hist<0>, &d.prune_hist);
    resident(k_prune_hist<1>, &d.prune_hist);
    resident(k_prune_hist<2>, &d.prune_hist);
    resident(k_prune_ties, &d.prune_hist);
    resident(k_prune_write, &d.prune_write);
    resident(k_prune_write_ranked, &d.prune_write_ranked);
    if (e == cudaSuccess && (d.sumsq < 1 || d.feedback_add < 1 || d.prune_hist < 1 || d.prune_write < 1 || d.prune_write_ranked < 1)) e = cudaErrorUnknown;
    int coop = 0;
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev);
    if (e != cudaSuccess || d.compact_feedback < 1 || d.finalize_small < 1 || d.finalize_large < 1 || d.merge < 1 || !coop) {
      cudaGetLastError();
      return NSML_ERR_CUDA;
    }
    d.ready = true;
  }
  *out = &d;
  return NSML_OK;
}

static inline bool valid_bits(int bits) { return bits == NSML_BITS_INT8 || bits == NSML_BITS_FP16 || bits == NSML_BITS_FP32; }
static inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

static inline unsigned int grid_for(unsigned long long work_items, unsigned long long per_block, int cap) {
  unsigned long long blocks = (work_items + per_block - 1) / per_block;
  if (blocks < 1) blocks = 1;
  if (blocks > (unsigned long long)cap) blocks = cap;
  return (unsigned int)blocks;
}

// The short, latency-bound kernels (sample, gather, list stage, partition) are launched at the highest stream
// priority.  When several buckets are in flight on several streams, every bucket pass that is ready sits in
// front of the device's block scheduler with thousands of blocks to place; a list-stage kernel that becomes
// ready later is otherwise placed only after all of them, so the passes of a step ran first, back to back,
// and the list stages afterwards with nothing to overlap them (measured with a timer in every kernel:
// 250 us of an 800 us step).  At high priority its few blocks are placed as soon as blocks of the running pass
// retire, and it runs beside the next pass.
static int high_priority() {
  static const int p = [] {
    int least = 0, greatest = 0;
    return cudaDeviceGetStreamPriorityRange(&least, &greatest) == cudaSuccess ? greatest : 0;
  }();
  return p;
}

template <class... KArgs, class... Args>
static cudaError_t launch_prio(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, bool cooperative,
                               unsigned int cluster_x, bool high, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[3];
  unsigned int na = 0;
  attr[na].id = cudaLaunchAttributePriority;
  attr[na].val.priority = high ? high_priority() : 0;
  ++na;
  if (cooperative) {
    attr[na].id = cudaLaunchAttributeCooperative;
    attr[na].val.cooperative = 1;
    ++na;
  }
  if (cluster_x) {
    attr[na].id = cudaLaunchAttributeClusterDimension;
    attr[na].val.clusterDim.x = cluster_x;
    attr[na].val.clusterDim.y = 1;
    attr[na].val.clusterDim.z = 1;
    ++na;
  }
  cfg.attrs = attr;
  cfg.numAttrs = na;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

static int64_t k_of(int64_t n, double ratio) {
  if (n < 1 || n > NSML_MAX_N || !(ratio > 0.0) || !(ratio <= 1.0)) return 0;
  double kd = std::ceil(ratio * (double)n);
  int64_t k = (int64_t)kd;
  if (k < 1) k = 1;
  if (k > n) k = n;
  return k;
}

// Rank (from the top, 1-based) of the sample key that becomes the bracket's
// lower bound: the expected rank of the k-th largest among kSamples draws plus
// six standard deviations.  0 = do not sample (small bucket, or nearly
// everything is kept): the bracket then starts at key 0.
static unsigned int sample_rank(int64_t n, int64_t k) {
  if (n < 2 * (int64_t)kSamples) return 0;
  const double p = (double)k / (double)n;
  const double j = std::ceil(kSamples * p + 6.0 * std::sqrt(kSamples * p * (1.0 - p))) + 1.0;
  if (j >= (double)kSamples) return 0;
  return (unsigned int)j;
}

// Candidates per block of the list stage's small shape (nsml_set_list_block_candidates).
static std::atomic<int> g_list_block_candidates{4096};

// Kept fraction from which the select runs over the bucket itself.
constexpr double kDenseRatioAny = 0.25;

static unsigned long long finalize_large_blocks(const DeviceInfo& dev) {
  return (unsigned long long)dev.sms * (dev.finalize_large < 2 ? dev.finalize_large : 2);
}

// Dense mode: the finalize kernel selects over the bucket itself, with no sample and no bucket pass.
// Taken when the bucket cannot be sampled and when the candidate list (8 bytes per entry) would be about
// as large as the bucket.
static bool use_dense(int64_t n, int64_t k, const DeviceInfo&) {
  const double p_keep = (double)k / (double)n;
  return sample_rank(n, k) == 0 || p_keep >= kDenseRatioAny;
}

// DTYPE: element type of `grad` (what the sample and the bucket pass read).  FDTYPE: element type of the
// bucket the later stages re-read; with a residual (local accumulation fused into the bucket pass, list
// strategy only) that bucket is the residual buffer, float32, which then holds gradient + residual.
template <int DTYPE, int FDTYPE>
static int launch_compress(const void* grad, float* residual, const uint32_t* mask, int64_t n, int64_t k, int bits,
                           unsigned char* ws, unsigned char* payload, const CompressLayout& L, const PayloadLayout& P,
                           const DeviceInfo& dev, cudaStream_t st, bool keep_status = false) {
  Ctl* ctl = reinterpret_cast<Ctl*>(ws);
  unsigned short* seg_off = reinterpret_cast<unsigned short*>(ws + L.seg_off);
  uint32_t* seg_val = reinterpret_cast<uint32_t*>(ws + L.seg_val);
  unsigned short* seg_count = reinterpret_cast<unsigned short*>(ws + L.seg_count);
  const unsigned long long nseg = ((unsigned long long)n + kSegElems - 1) / kSegElems;
  BucketSrc<DTYPE> src{grad, mask};
  BucketSrc<FDTYPE> fsrc{residual != nullptr ? static_cast<const void*>(residual) : grad, mask};
  const double p_keep = (double)k / (double)n;
  const unsigned long long large_cap_blocks = finalize_large_blocks(dev);
  const bool dense = use_dense(n, k, dev);
  unsigned int fgrid;
  bool small_shape;
  bool cluster_shape = false;
  if (dense) {
    small_shape = (unsigned long long)n <= (unsigned long long)dev.sms * kFinSmallCache;
    unsigned long long cap = small_shape ? (unsigned long long)dev.sms : large_cap_blocks;
    if (cap > (unsigned long long)kMaxFinalizeBlocks) cap = kMaxFinalizeBlocks;
    unsigned long long want = (unsigned long long)n / 4096 + 1;  // at least about 4096 elements per block
    if (want > nseg) want = nseg;
    fgrid = (unsigned int)(want < cap ? want : cap);
    LaunchScope scope(K_CLEAR, st);
    k_clear<<<4, kCta, 0, st>>>(reinterpret_cast<uint4*>(ws), (unsigned int)(L.group_count / 16), keep_status ? 1 : 0);
  } else {
    {
      LaunchScope scope(K_SAMPLE, st);  // one cluster of kSampleBlocks blocks
      // (the cluster shape is part of the kernel's definition)
      launch_prio(k_sample<DTYPE>, dim3(kSampleBlocks), dim3(kSampleThreads), 0, st, false, 0, true, src, residual, (unsigned long long)n,
                  sample_rank(n, k), ctl, reinterpret_cast<uint4*>(ws), (unsigned int)(L.zero_bytes / 16), keep_status ? 1 : 0);
    }
    {
      // bucket pass.  With a residual: persistent blocks, a block takes 8 segments per step, at most 4
      // resident blocks per SM.  Without: a warp per 2 KB of the bucket, eight warps per block.
      LaunchScope scope(K_COMPACT_BUCKET, st);
      const int resident = dev.compact_feedback;
      const int per_sm = resident < 4 ? resident : 4;
      constexpr unsigned long long kPlainSegs = (kCta / 32) * compact_segs_per_warp<DTYPE>();  // segments per block
      const unsigned int grid = residual != nullptr ? grid_for(nseg, kCta / 32, dev.sms * per_sm)
                                                    : (unsigned int)((nseg + kPlainSegs - 1) / kPlainSegs);
      unsigned int* group_count = reinterpret_cast<unsigned int*>(ws + L.group_count);
      if (residual != nullptr)
        k_compact_bucket<DTYPE, true><<<grid, kCta, kCompactFeedbackSmem, st>>>(src, residual, (unsigned long long)n, ctl, seg_off,
                                                                                seg_val, seg_count, group_count);
      else if (mask != nullptr)
        k_compact_bucket<DTYPE, false, true><<<grid, kCta, 0, st>>>(src, nullptr, (unsigned long long)n, ctl, seg_off, seg_val,
                                                                    seg_count, group_count);
      else
        k_compact_bucket<DTYPE, false, false><<<grid, kCta, 0, st>>>(src, nullptr, (unsigned long long)n, ctl, seg_off, seg_val,
                                                                     seg_count, group_count);
    }
    // list stage: cooperative, every block co-resident.  The small shape when a block's share of the
    // expected candidates (k plus the sampling margin) fits its shared-memory cache.
    fgrid = (unsigned int)dev.sms;
    if ((unsigned long long)fgrid > nseg) fgrid = (unsigned int)nseg;
    if (fgrid > (unsigned int)kMaxFinalizeBlocks) fgrid = kMaxFinalizeBlocks;
    const double expected = (double)n * (p_keep + 6.0 * std::sqrt(p_keep * (1.0 - p_keep) / kSamples)) + 64.0;
    small_shape = expected / fgrid <= (double)kFinSmallCache;
    cluster_shape = dev.finalize_cluster && expected <= kFinClusterMaxCandidates && nseg >= (unsigned long long)kFinClusterBlocks;
    if (cluster_shape) {
      fgrid = kFinClusterBlocks;
    } else if (small_shape) {  // short lists: no more blocks than about 4096 candidates each (cheaper barriers, one block = none)
      unsigned int want = (unsigned int)(expected / (double)g_list_block_candidates.load(std::memory_order_relaxed)) + 1;
      if (want < fgrid) fgrid = want;
    } else {  // long lists: as many blocks as stay co-resident (two per SM)
      unsigned long long cap = large_cap_blocks;
      // (a caller that asked for few, long list-stage blocks gets one per SM while a block's share still fits its cache)
      if (g_list_block_candidates.load(std::memory_order_relaxed) > 4096 && expected / dev.sms <= (double)kFinLargeCache)
        cap = (unsigned long long)dev.sms;
      if (cap > nseg) cap = nseg;
      if (cap > (unsigned long long)kMaxFinalizeBlocks) cap = kMaxFinalizeBlocks;
      if (cap > fgrid) fgrid = (unsigned int)cap;
    }
  }
  FinalizeParams fp;
  fp.n = (unsigned long long)n;
  fp.k = (unsigned long long)k;
  fp.bits = bits;
  fp.nseg = nseg;
  fp.ctl = ctl;
  fp.hist = reinterpret_cast<unsigned int*>(ws + L.hist);
  fp.block_counts = reinterpret_cast<unsigned long long*>(ws + L.block_counts);
  fp.seg_count = seg_count;
  fp.group_count = reinterpret_cast<const unsigned int*>(ws + L.group_count);
  fp.seg_off = seg_off;
  fp.seg_val = seg_val;
  fp.list_idx = reinterpret_cast<uint32_t*>(ws + L.list_idx);
  fp.list_val = reinterpret_cast<uint32_t*>(ws + L.list_val);
  fp.raw_val = reinterpret_cast<float*>(ws + L.raw_val);
  fp.payload = payload;
  fp.P = P;
  if (!dense) {
    LaunchScope scope(K_GATHER, st);  // segmented list -> contiguous list and the histogram of the first digit
    // blocks per group: about 1024 expected candidates (one step of the copy loop) per block, at least two
    // (candidates crowd into parts of a bucket), at most eight
    const unsigned long long ngroups = (nseg + kGatherSegs - 1) / kGatherSegs;
    const double per_group = (double)n * (p_keep + 6.0 * std::sqrt(p_keep * (1.0 - p_keep) / kSamples)) / (double)ngroups;
    unsigned int split = (unsigned int)(per_group / 1024.0) + 1;
    // (with more than the default candidates per list-stage block the caller has asked for few, long blocks: one
    // gather block per group then, 21 instead of 16 us alone, 2-3 % more throughput with eight streams)
    const unsigned int min_split = g_list_block_candidates.load(std::memory_order_relaxed) > 4096 ? 1u : 2u;
    split = split < min_split ? min_split : (split > 8 ? 8 : split);
    launch_prio(k_gather, dim3((unsigned int)(ngroups * split)), dim3(kGatherThreads), 0, st, false, 0, true, fp, split);
  }
  {
    LaunchScope scope(dense ? K_FINALIZE_DENSE : K_FINALIZE, st);
    cudaError_t le;
    auto launch = [&](auto kernel, int threads, int cache) {  // cooperative: every block co-resident
      return launch_prio(kernel, dim3(fgrid), dim3(threads), finalize_dyn_smem(cache), st, true, 0, !dense, fsrc, fp);  // (the dense select streams the whole bucket: normal priority)
    };
    if (cluster_shape) {
      // one cluster; the blocks of a cluster are co-scheduled by the hardware, so no cooperative launch is needed
      le = launch_prio(k_finalize<FDTYPE, kFinClusterThreads, kFinClusterCache, true>, dim3(kFinClusterBlocks), dim3(kFinClusterThreads),
                       finalize_dyn_smem(kFinClusterCache), st, false, kFinClusterBlocks, true, fsrc, fp);
    } else if (small_shape && dense) le = launch(k_finalize_dense<FDTYPE, kFinSmallThreads, kFinSmallCache>, kFinSmallThreads, kFinSmallCache);
    else if (small_shape) le = launch(k_finalize<FDTYPE, kFinSmallThreads, kFinSmallCache>, kFinSmallThreads, kFinSmallCache);
    else if (dense) le = launch(k_finalize_dense<FDTYPE, kFinLargeThreads, kFinDenseLargeCache>, kFinLargeThreads, kFinDenseLargeCache);
    else le = launch(k_finalize<FDTYPE, kFinLargeThreads, kFinLargeCache>, kFinLargeThreads, kFinLargeCache);
    if (le != cudaSuccess) return NSML_ERR_CUDA;
  }
  return NSML_OK;
}

static int compress_impl(const void* grad, int64_t n, int grad_dtype, double ratio, int bits,
                         const uint32_t* prune_mask, void* payload, size_t payload_capacity, void* workspace,
                         size_t workspace_bytes, cudaStream_t st, bool keep_status = false) {
  if (grad == nullptr || payload == nullptr || workspace == nullptr) return NSML_ERR_ARG;
  if (grad_dtype != NSML_F32 && grad_dtype != NSML_BF16) return NSML_ERR_ARG;
  if (!valid_bits(bits)) return NSML_ERR_ARG;
  const int64_t k = k_of(n, ratio);
  if (k == 0) return NSML_ERR_ARG;
  if (!aligned(grad, 16) || !aligned(payload, 16) || !aligned(workspace, 256)) return NSML_ERR_ARG;
  if (prune_mask != nullptr && !aligned(prune_mask, 4)) return NSML_ERR_ARG;
  const PayloadLayout P = payload_layout(k, bits);
  const CompressLayout L = compress_layout(n);
  if (payload_capacity < P.total || workspace_bytes < L.total) return NSML_ERR_CAPACITY;
  const DeviceInfo* dev = nullptr;
  int rc = device_info(&dev);
  if (rc != NSML_OK) return rc;
  unsigned char* ws = static_cast<unsigned char*>(workspace);
  unsigned char* pl = static_cast<unsigned char*>(payload);
  if (grad_dtype == NSML_F32) rc = launch_compress<NSML_F32, NSML_F32>(grad, nullptr, prune_mask, n, k, bits, ws, pl, L, P, *dev, st, keep_status);
  else rc = launch_compress<NSML_BF16, NSML_BF16>(grad, nullptr, prune_mask, n, k, bits, ws, pl, L, P, *dev, st, keep_status);
  if (rc != NSML_OK) return rc;
  if (cudaGetLastError() != cudaSuccess) return NSML_ERR_CUDA;
  return NSML_OK;
}

// payload_bytes: sizes of the buffers behind the payload pointers, or nullptr when the caller does not
// know them.  timed: whether the launches may be bracketed by profiling events.
static int accumulate_impl(const void* const* payloads, const size_t* payload_bytes, int W, float* dense, int64_t n,
                           int zero_first, void* workspace, size_t workspace_bytes, cudaStream_t st, bool timed = true) {
  if (payloads == nullptr || dense == nullptr || workspace == nullptr) return NSML_ERR_ARG;
  if (W < 1 || W > NSML_MAX_WORKERS || n < 1 || n > NSML_MAX_N) return NSML_ERR_ARG;
  if (!aligned(dense, 16) || !aligned(workspace, 256)) return NSML_ERR_ARG;
  PayloadTable table;
  std::memset(&table, 0, sizeof(table));
  for (int w = 0; w < W; ++w) {
    if (payloads[w] == nullptr || !aligned(payloads[w], 16)) return NSML_ERR_ARG;
    table.p[w] = static_cast<const unsigned char*>(payloads[w]);
    if (payload_bytes != nullptr) {
      if (payload_bytes[w] < sizeof(nsml_payload_header)) return NSML_ERR_ARG;
      table.bytes[w] = payload_bytes[w];
    }
  }
  const AccumulateLayout L = accumulate_layout(n, W);
  if (workspace_bytes < L.total) return NSML_ERR_CAPACITY;
  const DeviceInfo* dev = nullptr;
  int rc = device_info(&dev);
  if (rc != NSML_OK) return rc;

  unsigned char* ws = static_cast<unsigned char*>(workspace);
  int* status = reinterpret_cast<int*>(ws);
  unsigned int* offsets = reinterpret_cast<unsigned int*>(ws + L.offsets);
  const unsigned int tiles = (unsigned int)((n + kDenseTile - 1) / kDenseTile);
  {
    LaunchScope scope(K_PARTITION, st, timed);  // also clears the status word
    const unsigned long long offsets_needed = (unsigned long long)W * (tiles + 1ull);
    if (offsets_needed <= 4096) {  // few offsets: a warp each, few round trips (from about ten thousand offsets on the
                                   // thread-per-offset form takes as long alone, 12.8 us, and leaves the SMs to other streams:
                                   // eight-stream step of the default workload 0.645 -> 0.626 ms)
      unsigned int grid = (unsigned int)((offsets_needed * 32 + kCta - 1) / kCta);
      launch_prio(k_partition, dim3(grid), dim3(kCta), 0, st, false, 0, true, table, W, (unsigned long long)n, tiles, offsets, status);
    } else {  // many offsets: a thread each
      unsigned int grid = (unsigned int)((offsets_needed + kCta - 1) / kCta);
      launch_prio(k_partition_wide, dim3(grid), dim3(kCta), 0, st, false, 0, true, table, W, (unsigned long long)n, tiles, offsets, status);
    }
  }
  {
    LaunchScope scope(K_MERGE, st, timed);
    unsigned int grid = grid_for(tiles, 1, dev->sms * dev->merge);
    k_merge<<<grid, kCta, 0, st>>>(table, W, dense, (unsigned long long)n, zero_first, tiles, offsets, status);
  }
  if (cudaGetLastError() != cudaSuccess) return NSML_ERR_CUDA;
  return NSML_OK;
}

// ---- Alg. 2 Step 1: L2 norm and gate ----------------------------------------
// Blocks of the streaming kernels of nsml_adaptive.cuh: enough to keep every SM's loads in flight.
static unsigned int stream_grid(int64_t n, const DeviceInfo& dev, int per_sm, unsigned int cap) {
  unsigned int g = grid_for(((unsigned long long)n + kStreamTile - 1) / kStreamTile, 1, dev.sms * per_sm);
  return g < cap ? g : cap;
}

static int sumsq_impl(const void* grad, int64_t n, int grad_dtype, void* workspace, size_t workspace_bytes,
                      cudaStream_t st) {
  if (grad == nullptr || workspace == nullptr) return NSML_ERR_ARG;
  if (grad_dtype != NSML_F32 && grad_dtype != NSML_BF16) return NSML_ERR_ARG;
  if (n < 1 || n > NSML_MAX_N) return NSML_ERR_ARG;
  if (!aligned(grad, 16) || !aligned(workspace, 256)) return NSML_ERR_ARG;
  if (workspace_bytes < kSumsqWorkspace) return NSML_ERR_CAPACITY;
  const DeviceInfo* dev = nullptr;
  int rc = device_info(&dev);
  if (rc != NSML_OK) return rc;
  unsigned char* ws = static_cast<unsigned char*>(workspace);
  if (cudaMemsetAsync(ws, 0, 256, st) != cudaSuccess) return NSML_ERR_CUDA;
  SumsqCtl* ctl = reinterpret_cast<SumsqCtl*>(ws);
  double* partials = reinterpret_cast<double*>(ws + 256);
  const unsigned int grid = stream_grid(n, *dev, dev->sumsq < 8 ? dev->sumsq : 8, kSumsqMaxBlocks);
  {
    LaunchScope scope(K_SUMSQ, st);
    if (grad_dtype == NSML_F32)
      k_sumsq<NSML_F32><<<grid, kCta, 0, st>>>(BucketSrc<NSML_F32>{grad, nullptr}, (unsigned long long)n, ctl, partials);
    else
      k_sumsq<NSML_BF16><<<grid, kCta, 0, st>>>(BucketSrc<NSML_BF16>{grad, nullptr}, (unsigned long long)n, ctl, partials);
  }
  if (cudaGetLastError() != cudaSuccess) return NSML_ERR_CUDA;
  return NSML_OK;
}

// Synchronises the stream and reads the status word and the sum of squares left by sumsq_impl.
static int sumsq_read(const void* workspace, cudaStream_t st, double* sumsq) {
  SumsqCtl host;
  if (cudaMemcpyAsync(&host, workspace, sizeof(host), cudaMemcpyDeviceToHost, st) != cudaSuccess) return NSML_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return NSML_ERR_CUDA;
  if (host.status != NSML_OK) return host.status;
  *sumsq = host.sumsq;
  return NSML_OK;
}

static int gate(double ratio, double l2, double tr_q, double tr_d, int plain_bits, double* ratio_out, int* bits_out) {
  if (!(ratio > 0.0) || !(ratio <= 1.0) || !valid_bits(plain_bits) || !(l2 >= 0.0) || tr_q != tr_q || tr_d != tr_d)
    return NSML_ERR_ARG;
  if (ratio < tr_q && l2 > tr_d) {
    const double doubled = 2.0 * ratio;
    *ratio_out = doubled < 1.0 ? doubled : 1.0;
    *bits_out = NSML_BITS_FP16;
  } else {
    *ratio_out = ratio;
    *bits_out = plain_bits;
  }
  return NSML_OK;
}

// ---- Alg. 2 Step 2: pruning mask from the weights ---------------------------
static int64_t pruned_count(int64_t n, double ratio) {
  if (n < 1 || n > NSML_MAX_N || !(ratio > 0.0) || !(ratio <= 1.0)) return -1;
  const double rate = 0.5 * (1.0 - ratio);
  int64_t m = (int64_t)std::ceil(rate * (double)n);
  if (m < 0) m = 0;
  if (m > n) m = n;
  return m;
}

static int prune_impl(const float* weights, int64_t n, double ratio, uint32_t* mask, void* workspace,
                      size_t workspace_bytes, cudaStream_t st) {
  if (weights == nullptr || mask == nullptr || workspace == nullptr) return NSML_ERR_ARG;
  const int64_t m = pruned_count(n, ratio);
  if (m < 0) return NSML_ERR_ARG;
  if (!aligned(weights, 16) || !aligned(mask, 4) || !aligned(workspace, 256)) return NSML_ERR_ARG;
  const PruneLayout L = prune_layout(n);
  if (workspace_bytes < L.total) return NSML_ERR_CAPACITY;
  const DeviceInfo* dev = nullptr;
  int rc = device_info(&dev);
  if (rc != NSML_OK) return rc;
  unsigned char* ws = static_cast<unsigned char*>(workspace);
  if (cudaMemsetAsync(ws, 0, L.tie_list, st) != cudaSuccess) return NSML_ERR_CUDA;  // status, ctl, histograms
  if (m == 0) {  // ratio 1: nothing is pruned
    if (cudaMemsetAsync(mask, 0, (size_t)((n + 31) / 32) * 4, st) != cudaSuccess) return NSML_ERR_CUDA;
    return NSML_OK;
  }
  PruneCtl* ctl = reinterpret_cast<PruneCtl*>(ws);
  unsigned int* hist = reinterpret_cast<unsigned int*>(ws + L.hist);
  unsigned int* tile_ties = reinterpret_cast<unsigned int*>(ws + L.tile_ties);
  uint2* tie_list = reinterpret_cast<uint2*>(ws + L.tie_list);
  const BucketSrc<NSML_F32> src{weights, nullptr};
  const unsigned int grid = stream_grid(n, *dev, dev->prune_hist < 8 ? dev->prune_hist : 8, 1u << 16);
  const unsigned int wgrid = stream_grid(n, *dev, dev->prune_write < 8 ? dev->prune_write : 8, 1u << 16);
  const unsigned long long un = (unsigned long long)n;
  bool two_pass = false;
  // Two passes where a sample can bracket the threshold: ranks (from the top, among the complemented keys of
  // kPruneSamples weights) six standard deviations either side of the expected rank of the m-th largest.
  if (n >= 2 * (int64_t)kPruneSamples) {
    const double p = (double)m / (double)n, mean = kPruneSamples * p, six = 6.0 * std::sqrt(kPruneSamples * p * (1.0 - p));
    const double r_lo = std::ceil(mean + six) + 1.0, r_hi = std::floor(mean - six);
    if (r_lo < (double)kPruneSamples && r_hi >= 1.0) {
      two_pass = true;
      unsigned int* fine = reinterpret_cast<unsigned int*>(ws + L.fine);
      {
        LaunchScope scope(K_PRUNE_SAMPLE, st);
        launch_prio(k_prune_sample, dim3(1), dim3(1024), 0, st, false, 0, true, src, un, (unsigned int)r_lo, (unsigned int)r_hi, ctl);
      }
      {
        LaunchScope scope(K_PRUNE_COUNT, st);
        k_prune_count<<<grid, kCta, 0, st>>>(src, un, ctl, fine);
      }
      {
        LaunchScope scope(K_PRUNE_SETTLE, st);
        launch_prio(k_prune_settle, dim3(1), dim3(kCta), 0, st, false, 0, true, (unsigned int)m, ctl, fine);
      }
      {
        LaunchScope scope(K_PRUNE_MARK, st);
        // a block per 16 KB tile: short-lived blocks on one moving window read faster than persistent ones
        const unsigned long long mark_tiles = (un + kStreamTile - 1) / kStreamTile;
        k_prune_mark<<<(unsigned int)mark_tiles, kCta, 0, st>>>(src, un, ctl, tie_list, mask);
      }
      {
        LaunchScope scope(K_PRUNE_FIX, st);
        launch_prio(k_prune_fix, dim3(kPruneFixBlocks), dim3(kCta), 0, st, false, 0, true, ctl, tie_list, mask);
      }
    }
  }
  // The four-pass build: every kernel of it leaves at once when the two passes above have built the mask.  Behind
  // the two-pass path it is the rare fallback, so it gets small grids (two blocks per SM): what counts there is
  // how little the six launches cost when they have nothing to do; they are then launched at high priority
  // like the other short kernels, so that they do not queue behind other streams' passes.
  const unsigned int small = (unsigned int)dev->sms * 2;
  const unsigned int fgrid = two_pass && grid > small ? small : grid;
  const unsigned int fwgrid = two_pass && wgrid > small ? small : wgrid;
  {
    LaunchScope scope(K_PRUNE_HIST, st);
    launch_prio(k_prune_hist<0>, dim3(fgrid), dim3(kCta), 0, st, false, 0, two_pass, src, un, (unsigned int)m, ctl, hist, tie_list);
  }
  {
    LaunchScope scope(K_PRUNE_HIST, st);
    launch_prio(k_prune_hist<1>, dim3(fgrid), dim3(kCta), 0, st, false, 0, two_pass, src, un, (unsigned int)m, ctl, hist, tie_list);
  }
  {
    LaunchScope scope(K_PRUNE_HIST, st);
    launch_prio(k_prune_hist<2>, dim3(fgrid), dim3(kCta), 0, st, false, 0, two_pass, src, un, (unsigned int)m, ctl, hist, tie_list);
  }
  {
    LaunchScope scope(K_PRUNE_TIES, st);
    launch_prio(k_prune_ties, dim3(fgrid), dim3(kCta), 0, st, false, 0, two_pass, src, un, ctl, hist, tie_list, tile_ties);
  }
  {
    LaunchScope scope(K_PRUNE_WRITE, st);
    launch_prio(k_prune_write, dim3(fwgrid), dim3(kCta), 0, st, false, 0, two_pass, src, un, ctl, tile_ties, mask);
  }
  {
    LaunchScope scope(K_PRUNE_WRITE_RANKED, st);  // returns at once unless ties have to be ranked
    unsigned int rgrid = stream_grid(n, *dev, dev->prune_write_ranked < 8 ? dev->prune_write_ranked : 8, 1u << 16);
    if (two_pass && rgrid > small) rgrid = small;
    launch_prio(k_prune_write_ranked, dim3(rgrid), dim3(kCta), 0, st, false, 0, two_pass, src, un, ctl, tile_ties, mask);
  }
  if (cudaGetLastError() != cudaSuccess) return NSML_ERR_CUDA;
  return NSML_OK;
}

// ---- Section 4.2 Step 3: local accumulation of the filtered gradients ---------
static int feedback_impl(const void* grad, float* residual, int64_t n, int grad_dtype, double ratio, int bits,
                         const uint32_t* prune_mask, void* payload, size_t payload_capacity, void* workspace,
                         size_t workspace_bytes, cudaStream_t st) {
  if (grad == nullptr || residual == nullptr) return NSML_ERR_ARG;
  if (grad_dtype != NSML_F32 && grad_dtype != NSML_BF16) return NSML_ERR_ARG;
  const int64_t k = k_of(n, ratio);
  if (k == 0 || !valid_bits(bits)) return NSML_ERR_ARG;
  if (!aligned(grad, 16) || !aligned(residual, 16)) return NSML_ERR_ARG;
  if (payload == nullptr || workspace == nullptr || !aligned(payload, 16) || !aligned(workspace, 256)) return NSML_ERR_ARG;
  if (payload_capacity < payload_layout(k, bits).total || workspace_bytes < compress_layout(n).total)
    return NSML_ERR_CAPACITY;
  const DeviceInfo* dev = nullptr;
  int rc = device_info(&dev);
  if (rc != NSML_OK) return rc;
  if (use_dense(n, k, *dev)) {
    // dense strategy (no bucket pass to fuse the add into): residual <- grad + residual first, then the select
    // over the residual buffer
    const unsigned int grid = stream_grid(n, *dev, dev->feedback_add < 8 ? dev->feedback_add : 8, 1u << 16);
    {
      LaunchScope scope(K_FEEDBACK_ADD, st);
      if (grad_dtype == NSML_F32)
        k_feedback_add<NSML_F32><<<grid, kCta, 0, st>>>(BucketSrc<NSML_F32>{grad, nullptr}, residual, (unsigned long long)n);
      else
        k_feedback_add<NSML_BF16><<<grid, kCta, 0, st>>>(BucketSrc<NSML_BF16>{grad, nullptr}, residual, (unsigned long long)n);
    }
    rc = compress_impl(residual, n, NSML_F32, ratio, bits, prune_mask, payload, payload_capacity, workspace,
                       workspace_bytes, st);
  } else {
    // list strategy: the bucket pass adds the residual as it streams the gradient and leaves the sum in it
    if (prune_mask != nullptr && !aligned(prune_mask, 4)) return NSML_ERR_ARG;
    unsigned char* ws = static_cast<unsigned char*>(workspace);
    unsigned char* pl = static_cast<unsigned char*>(payload);
    const PayloadLayout P = payload_layout(k, bits);
    const CompressLayout L = compress_layout(n);
    if (grad_dtype == NSML_F32)
      rc = launch_compress<NSML_F32, NSML_F32>(grad, residual, prune_mask, n, k, bits, ws, pl, L, P, *dev, st);
    else
      rc = launch_compress<NSML_BF16, NSML_F32>(grad, residual, prune_mask, n, k, bits, ws, pl, L, P, *dev, st);
  }
  if (rc != NSML_OK) return rc;
  {
    LaunchScope scope(K_FEEDBACK_SUBTRACT, st);
    const unsigned int sgrid = grid_for((unsigned long long)k, kCta, dev->sms * 8);
    k_feedback_subtract<<<sgrid, kCta, 0, st>>>(static_cast<const unsigned char*>(payload), residual,
                                                (unsigned long long)n, static_cast<int*>(workspace));
  }
  if (cudaGetLastError() != cudaSuccess) return NSML_ERR_CUDA;
  return NSML_OK;
}

// ---- scratch for nsml_decompress_accumulate_static --------------------------
// Part of the library image: every device that loads the library holds this
// array until exit.  In host code the name below is only a handle; the device
// address is looked up once per device with cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_static_scratch[NSML_STATIC_SCRATCH_BYTES];

static void* g_static_scratch_addr[64];
static std::mutex g_static_mutex;

static int static_scratch(void** out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return NSML_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_static_mutex);
  if (g_static_scratch_addr[dev] == nullptr) {
    void* addr = nullptr;
    if (cudaGetSymbolAddress(&addr, g_static_scratch) != cudaSuccess || addr == nullptr) {
      cudaGetLastError();
      return NSML_ERR_CUDA;
    }
    g_static_scratch_addr[dev] = addr;
  }
  *out = g_static_scratch_addr[dev];
  return NSML_OK;
}

}  // namespace nsml

using namespace nsml;

extern "C" {

int64_t nsml_k_of(int64_t n, double ratio) { return k_of(n, ratio); }

int nsml_compress_strategy(int64_t n, double ratio) {
  const int64_t k = k_of(n, ratio);
  if (k == 0) return NSML_ERR_ARG;
  const DeviceInfo* dev = nullptr;
  const int rc = device_info(&dev);
  if (rc != NSML_OK) return rc;
  return use_dense(n, k, *dev) ? NSML_STRATEGY_DENSE : NSML_STRATEGY_LIST;
}

int nsml_set_list_block_candidates(int candidates) {
  if (candidates < 1024 || candidates > kFinSmallCache) return NSML_ERR_ARG;
  g_list_block_candidates.store(candidates, std::memory_order_relaxed);
  return NSML_OK;
}

size_t nsml_payload_bytes(int64_t n, double ratio, int bits) {
  if (!valid_bits(bits)) return 0;
  const int64_t k = k_of(n, ratio);
  if (k == 0) return 0;
  return payload_layout(k, bits).total;
}

size_t nsml_workspace_bytes(int64_t n, int grad_dtype) {
  if (n < 1 || n > NSML_MAX_N || (grad_dtype != NSML_F32 && grad_dtype != NSML_BF16)) return 0;
  return compress_layout(n).total;
}

size_t nsml_accumulate_workspace_bytes(int64_t n, int W) {
  if (n < 1 || n > NSML_MAX_N || W < 1 || W > NSML_MAX_WORKERS) return 0;
  return accumulate_layout(n, W).total;
}

int nsml_compress(const void* grad, int64_t n, int grad_dtype, double ratio, int bits, const uint32_t* prune_mask,
                  void* payload, size_t payload_capacity, void* workspace, size_t workspace_bytes, void* stream) {
  return compress_impl(grad, n, grad_dtype, ratio, bits, prune_mask, payload, payload_capacity, workspace,
                       workspace_bytes, static_cast<cudaStream_t>(stream));
}

int nsml_decompress_accumulate(const void* const* payloads, int W, float* dense, int64_t n, int zero_first,
                               void* workspace, size_t workspace_bytes, void* stream) {
  return accumulate_impl(payloads, nullptr, W, dense, n, zero_first, workspace, workspace_bytes,
                         static_cast<cudaStream_t>(stream));
}

int nsml_decompress_accumulate_sized(const void* const* payloads, const size_t* payload_bytes, int W, float* dense,
                                     int64_t n, int zero_first, void* workspace, size_t workspace_bytes, void* stream) {
  if (payload_bytes == nullptr) return NSML_ERR_ARG;
  return accumulate_impl(payloads, payload_bytes, W, dense, n, zero_first, workspace, workspace_bytes,
                         static_cast<cudaStream_t>(stream));
}

int nsml_decompress_accumulate_static(const void* const* payloads, int W, float* dense, int64_t n, int zero_first,
                                      void* stream, int* status_out) {
  if (n > NSML_STATIC_MAX_N || W > NSML_STATIC_MAX_WORKERS) return NSML_ERR_CAPACITY;
  if (n < 1 || W < 1) return NSML_ERR_ARG;
  if (accumulate_layout(n, W).total > (size_t)NSML_STATIC_SCRATCH_BYTES) return NSML_ERR_CAPACITY;
  void* scratch = nullptr;
  int rc = static_scratch(&scratch);
  if (rc != NSML_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  rc = accumulate_impl(payloads, nullptr, W, dense, n, zero_first, scratch, NSML_STATIC_SCRATCH_BYTES, st, /*timed=*/false);
  if (rc != NSML_OK || status_out == nullptr) return rc;
  int value = 0;
  if (cudaMemcpyAsync(&value, scratch, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return NSML_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return NSML_ERR_CUDA;
  *status_out = value;
  return NSML_OK;
}

// ---- Alg. 2 Steps 1-2 and the local accumulation of Step 3 --------------------
size_t nsml_l2_workspace_bytes(void) { return kSumsqWorkspace; }

int nsml_grad_l2(const void* grad, int64_t n, int grad_dtype, void* workspace, size_t workspace_bytes, void* stream,
                 double* l2_out) {
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int rc = sumsq_impl(grad, n, grad_dtype, workspace, workspace_bytes, st);
  if (rc != NSML_OK || l2_out == nullptr) return rc;
  double sumsq = 0.0;
  rc = sumsq_read(workspace, st, &sumsq);
  if (rc != NSML_OK) return rc;
  *l2_out = std::sqrt(sumsq);
  return NSML_OK;
}

int nsml_quantize_gate(double ratio, double l2, double tr_q, double tr_d, int plain_bits, double* ratio_out,
                       int* bits_out) {
  if (ratio_out == nullptr || bits_out == nullptr) return NSML_ERR_ARG;
  return gate(ratio, l2, tr_q, tr_d, plain_bits, ratio_out, bits_out);
}

int64_t nsml_pruned_count(int64_t n, double ratio) {
  const int64_t m = pruned_count(n, ratio);
  return m < 0 ? 0 : m;
}

size_t nsml_prune_workspace_bytes(int64_t n) {
  if (n < 1 || n > NSML_MAX_N) return 0;
  return prune_layout(n).total;
}

int nsml_prune_mask_build(const float* weights, int64_t n, double ratio, uint32_t* prune_mask, void* workspace,
                          size_t workspace_bytes, void* stream) {
  return prune_impl(weights, n, ratio, prune_mask, workspace, workspace_bytes, static_cast<cudaStream_t>(stream));
}

int nsml_compress_feedback(const void* grad, float* residual, int64_t n, int grad_dtype, double ratio, int bits,
                           const uint32_t* prune_mask, void* payload, size_t payload_capacity, void* workspace,
                           size_t workspace_bytes, void* stream) {
  return feedback_impl(grad, residual, n, grad_dtype, ratio, bits, prune_mask, payload, payload_capacity, workspace,
                       workspace_bytes, static_cast<cudaStream_t>(stream));
}

size_t nsml_adaptive_payload_bytes(int64_t n, double ratio, double tr_q, int plain_bits) {
  size_t need = nsml_payload_bytes(n, ratio, plain_bits);
  if (need == 0) return 0;
  if (ratio < tr_q) {
    const double doubled = 2.0 * ratio;
    const size_t q = nsml_payload_bytes(n, doubled < 1.0 ? doubled : 1.0, NSML_BITS_FP16);
    if (q > need) need = q;
  }
  return need;
}

size_t nsml_adaptive_workspace_bytes(int64_t n, int grad_dtype) {
  size_t need = nsml_workspace_bytes(n, grad_dtype);
  if (need == 0) return 0;
  if (need < kSumsqWorkspace) need = kSumsqWorkspace;
  const size_t p = prune_layout(n).total;
  return need < p ? p : need;
}

int nsml_compress_adaptive(const void* grad, int64_t n, int grad_dtype, double ratio, double tr_q, double tr_d,
                           int plain_bits, const float* weights, uint32_t* prune_mask, void* payload,
                           size_t payload_capacity, void* workspace, size_t workspace_bytes, void* stream,
                           double* ratio_used, int* bits_used, double* l2_out) {
  if (ratio_used == nullptr || bits_used == nullptr) return NSML_ERR_ARG;
  if (!(ratio > 0.0) || !(ratio <= 1.0) || !valid_bits(plain_bits) || tr_q != tr_q || tr_d != tr_d) return NSML_ERR_ARG;
  if (weights != nullptr && prune_mask == nullptr) return NSML_ERR_ARG;
  const size_t need_ws = nsml_adaptive_workspace_bytes(n, grad_dtype);
  if (need_ws == 0) return NSML_ERR_ARG;
  if (workspace_bytes < need_ws) return NSML_ERR_CAPACITY;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // Step 1: the norm is needed only when the ratio is below the quantisation check threshold
  double use_ratio = ratio, l2 = -1.0;
  int use_bits = plain_bits;
  if (ratio < tr_q) {
    int rc = sumsq_impl(grad, n, grad_dtype, workspace, workspace_bytes, st);
    if (rc != NSML_OK) return rc;
    double sumsq = 0.0;
    rc = sumsq_read(workspace, st, &sumsq);
    if (rc != NSML_OK) return rc;
    l2 = std::sqrt(sumsq);
    rc = gate(ratio, l2, tr_q, tr_d, plain_bits, &use_ratio, &use_bits);
    if (rc != NSML_OK) return rc;
  }
  if (l2_out != nullptr) *l2_out = l2;
  *ratio_used = use_ratio;
  *bits_used = use_bits;
  // Step 2: the mask follows the ratio Step 1 left
  if (weights != nullptr) {
    const int rc = prune_impl(weights, n, use_ratio, prune_mask, workspace, workspace_bytes, st);
    if (rc != NSML_OK) return rc;
  }
  // Step 3.  The mask build shares the workspace and its status word with this step: when it ran, the
  // word is kept instead of cleared, so that non-finite weights found in Step 2 are still reported.
  return compress_impl(grad, n, grad_dtype, use_ratio, use_bits, prune_mask, payload, payload_capacity, workspace,
                       workspace_bytes, st, /*keep_status=*/weights != nullptr);
}

// ---- host-buffer variants --------------------------------------------------
static size_t elem_size(int grad_dtype) { return grad_dtype == NSML_F32 ? 4 : 2; }

size_t nsml_compress_host_scratch_bytes(int64_t n, int grad_dtype, double ratio, int bits) {
  const size_t ws = nsml_workspace_bytes(n, grad_dtype);
  const size_t pb = nsml_payload_bytes(n, ratio, bits);
  if (ws == 0 || pb == 0) return 0;
  return align_up(ws, 256) + align_up((size_t)n * elem_size(grad_dtype), 256) +
         align_up((size_t)((n + 31) / 32) * 4, 256) + align_up(pb, 256);
}

int nsml_compress_host(const void* grad_host, int64_t n, int grad_dtype, double ratio, int bits,
                       const uint32_t* prune_mask_host, void* payload_host, size_t payload_capacity,
                       void* device_scratch, size_t scratch_bytes, void* stream) {
  if (grad_host == nullptr || payload_host == nullptr || device_scratch == nullptr) return NSML_ERR_ARG;
  const size_t need = nsml_compress_host_scratch_bytes(n, grad_dtype, ratio, bits);
  if (need == 0 || !aligned(device_scratch, 256)) return NSML_ERR_ARG;
  const size_t pb = nsml_payload_bytes(n, ratio, bits);
  if (scratch_bytes < need || payload_capacity < pb) return NSML_ERR_CAPACITY;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  unsigned char* base = static_cast<unsigned char*>(device_scratch);
  const size_t ws = align_up(nsml_workspace_bytes(n, grad_dtype), 256);
  const size_t gbytes = (size_t)n * elem_size(grad_dtype);
  const size_t mbytes = (size_t)((n + 31) / 32) * 4;
  unsigned char* d_grad = base + ws;
  unsigned char* d_mask = d_grad + align_up(gbytes, 256);
  unsigned char* d_payload = d_mask + align_up(mbytes, 256);
  if (cudaMemcpyAsync(d_grad, grad_host, gbytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return NSML_ERR_CUDA;
  if (prune_mask_host != nullptr &&
      cudaMemcpyAsync(d_mask, prune_mask_host, mbytes, cudaMemcpyHostToDevice, st) != cudaSuccess)
    return NSML_ERR_CUDA;
  int rc = compress_impl(d_grad, n, grad_dtype, ratio, bits,
                         prune_mask_host ? reinterpret_cast<const uint32_t*>(d_mask) : nullptr, d_payload, pb, base, ws,
                         st);
  if (rc != NSML_OK) return rc;
  if (cudaMemcpyAsync(payload_host, d_payload, pb, cudaMemcpyDeviceToHost, st) != cudaSuccess) return NSML_ERR_CUDA;
  return NSML_OK;
}

size_t nsml_accumulate_host_scratch_bytes(int64_t n, int W, size_t total_payload_bytes) {
  const size_t ws = nsml_accumulate_workspace_bytes(n, W);
  if (ws == 0) return 0;
  return align_up(ws, 256) + align_up((size_t)n * 4, 256) + total_payload_bytes + (size_t)W * 256;
}

int nsml_decompress_accumulate_host(const void* const* payloads_host, const size_t* payload_bytes, int W,
                                    float* dense_host, int64_t n, int zero_first, void* device_scratch,
                                    size_t scratch_bytes, void* stream) {
  if (payloads_host == nullptr || payload_bytes == nullptr || dense_host == nullptr || device_scratch == nullptr)
    return NSML_ERR_ARG;
  if (W < 1 || W > NSML_MAX_WORKERS || !aligned(device_scratch, 256)) return NSML_ERR_ARG;
  if (n < 1 || n > NSML_MAX_N) return NSML_ERR_ARG;
  size_t total = 0;
  for (int w = 0; w < W; ++w) {
    if (payloads_host[w] == nullptr || payload_bytes[w] < sizeof(nsml_payload_header)) return NSML_ERR_ARG;
    // (the headers are not looked at here: a payload may still be on its way into host memory, written by an
    // earlier asynchronous call on this stream; the device checks every header against payload_bytes[w])
    total += payload_bytes[w];
  }
  const size_t need = nsml_accumulate_host_scratch_bytes(n, W, total);
  if (need == 0) return NSML_ERR_ARG;
  if (scratch_bytes < need) return NSML_ERR_CAPACITY;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  unsigned char* base = static_cast<unsigned char*>(device_scratch);
  const size_t ws = align_up(nsml_accumulate_workspace_bytes(n, W), 256);
  float* d_dense = reinterpret_cast<float*>(base + ws);
  unsigned char* cursor = base + ws + align_up((size_t)n * 4, 256);
  const void* d_payloads[NSML_MAX_WORKERS];
  for (int w = 0; w < W; ++w) {
    if (cudaMemcpyAsync(cursor, payloads_host[w], payload_bytes[w], cudaMemcpyHostToDevice, st) != cudaSuccess)
      return NSML_ERR_CUDA;
    d_payloads[w] = cursor;
    cursor += align_up(payload_bytes[w], 256);
  }
  if (!zero_first &&
      cudaMemcpyAsync(d_dense, dense_host, (size_t)n * 4, cudaMemcpyHostToDevice, st) != cudaSuccess)
    return NSML_ERR_CUDA;
  int rc = accumulate_impl(d_payloads, payload_bytes, W, d_dense, n, zero_first, base, ws, st);
  if (rc != NSML_OK) return rc;
  if (cudaMemcpyAsync(dense_host, d_dense, (size_t)n * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return NSML_ERR_CUDA;
  return NSML_OK;
}

int nsml_last_status(const void* workspace, void* stream, int* status_out) {
  if (workspace == nullptr || status_out == nullptr) return NSML_ERR_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int value = 0;
  if (cudaMemcpyAsync(&value, workspace, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return NSML_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return NSML_ERR_CUDA;
  *status_out = value;
  return NSML_OK;
}

int nsml_selftest_bounded_wait(void* workspace, size_t workspace_bytes, int max_polls, void* stream) {
  if (workspace == nullptr || !aligned(workspace, 256) || max_polls < 1 || max_polls > (1 << 16)) return NSML_ERR_ARG;
  if (workspace_bytes < 256) return NSML_ERR_CAPACITY;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaMemsetAsync(workspace, 0, 256, st) != cudaSuccess) return NSML_ERR_CUDA;
  k_barrier_probe<<<2, 32, 0, st>>>(static_cast<Ctl*>(workspace), max_polls);
  if (cudaGetLastError() != cudaSuccess) return NSML_ERR_CUDA;
  return NSML_OK;
}

const char* nsml_strerror(int status) {
  switch (status) {
    case NSML_OK: return "ok";
    case NSML_ERR_ARG: return "bad argument (null or misaligned pointer, size or enum out of range)";
    case NSML_ERR_CAPACITY: return "payload buffer or workspace too small";
    case NSML_ERR_CUDA: return "a CUDA runtime call failed";
    case NSML_ERR_NONFINITE: return "the gradient bucket holds NaN or Inf";
    case NSML_ERR_TIMEOUT: return "a bounded wait between thread blocks ran out";
    case NSML_ERR_PAYLOAD: return "payload header or index out of range";
    case NSML_ERR_INTERNAL: return "internal invariant failed: survivor count differs from k";
    default: return "unknown status";
  }
}

// ---- instrumentation -------------------------------------------------------
int nsml_kernel_count(void) { return K_COUNT; }

const char* nsml_kernel_name(int kernel_id) {
  return (kernel_id >= 0 && kernel_id < K_COUNT) ? kKernelNames[kernel_id] : "";
}

int64_t nsml_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

int nsml_prof_enable(int on) {
  std::lock_guard<std::mutex> lock(g_prof_mutex);
  if (!on) {
    for (ProfRecord& r : g_prof_records) {
      cudaEventDestroy(r.start);
      cudaEventDestroy(r.stop);
    }
    g_prof_records.clear();
  }
  g_prof_on.store(on != 0, std::memory_order_relaxed);
  return NSML_OK;
}

int nsml_prof_read(int kernel_id, double* total_ms, int64_t* launches) {
  if (kernel_id < 0 || kernel_id >= K_COUNT || total_ms == nullptr || launches == nullptr) return NSML_ERR_ARG;
  std::lock_guard<std::mutex> lock(g_prof_mutex);
  prof_drain_locked();
  *total_ms = g_prof_ms[kernel_id];
  *launches = g_prof_launches[kernel_id];
  return NSML_OK;
}

int nsml_prof_reset(void) {
  std::lock_guard<std::mutex> lock(g_prof_mutex);
  prof_drain_locked();
  for (int i = 0; i < K_COUNT; ++i) {
    g_prof_ms[i] = 0.0;
    g_prof_launches[i] = 0;
  }
  return NSML_OK;
}

}  // extern "C"
