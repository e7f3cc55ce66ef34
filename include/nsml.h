/*
 * nsml.h -- C ABI of libnsml: the data-parallel hot path of NetSenseML's
 * adaptive compression phase on one NVIDIA B200 (sm_100a).
 *
 * Three operations, named after the paper's statement of the problem:
 *
 *   nsml_select_ratio            host   Alg. 1 (network status sensing and
 *                                       adaptive compression-ratio adjustment)
 *   nsml_compress                device Alg. 2 Steps 2-3 (apply the pruning
 *                                       mask, top-k sparsification at `ratio`)
 *                                       plus the value codec of Alg. 2 Step 1
 *   nsml_decompress_accumulate   device aggregation of the W gathered sparse
 *                                       payloads into one dense gradient
 *                                       (Section 4.2 Step 3; AllGather pattern
 *                                       of Section 5.3)
 *
 * `ratio` is the KEPT fraction, as in the paper (1 = send everything).
 *
 * Conventions
 *   - Every function returns NSML_OK (0) or a negative NSML_ERR_* code.  Nothing
 *     throws, aborts or traps.
 *   - "device pointer" = CUDA global memory of the current device, owned by the
 *     caller before and after the call.  "host pointer" = ordinary memory.
 *   - Device work is enqueued on `stream` (a cudaStream_t passed as void*, NULL
 *     = the default stream) and the call returns without synchronising.  The
 *     short, latency-bound kernels of a call (sample, gather, list stage,
 *     partition) are launched at the device's highest stream priority, whatever
 *     the priority of `stream`: with several buckets in flight on several
 *     streams they are then placed between the blocks of other buckets'
 *     streaming passes instead of behind them.  Order within `stream` is kept.
 *   - Argument errors are returned at once and enqueue nothing.  Errors that only
 *     the device can see (non-finite input, corrupt payload, a bounded wait that
 *     ran out) are written to a status word at the start of `workspace`; read it
 *     with nsml_last_status().
 *   - The library allocates no device memory: scratch comes in as `workspace`.
 *     Two calls that share a workspace must not overlap on the GPU.
 */
#ifndef NSML_H
#define NSML_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  NSML_OK = 0,
  NSML_ERR_ARG = -1,       /* NULL / misaligned pointer, size or enum out of range */
  NSML_ERR_CAPACITY = -2,  /* payload buffer or workspace too small */
  NSML_ERR_CUDA = -3,      /* a CUDA runtime call failed (no device, launch error) */
  NSML_ERR_NONFINITE = -4, /* device: the bucket holds NaN or Inf */
  NSML_ERR_TIMEOUT = -5,   /* device: a bounded wait between thread blocks ran out */
  NSML_ERR_PAYLOAD = -6,   /* device: payload header or index out of range */
  NSML_ERR_INTERNAL = -7   /* device: an internal invariant failed (survivor count != k) */
};

enum { NSML_F32 = 0, NSML_BF16 = 1 };              /* gradient element type */
enum { NSML_BITS_INT8 = 8, NSML_BITS_FP16 = 16, NSML_BITS_FP32 = 32 }; /* value codec ("bits") */

#define NSML_QBLOCK 1024         /* survivors per int8 scale block */
#define NSML_MAX_WORKERS 64      /* largest W of nsml_decompress_accumulate */
#define NSML_MAX_N 2147483647LL  /* largest bucket, elements */
#define NSML_PAYLOAD_MAGIC 0x4C4D534Eu /* "NSML" */
#define NSML_PAYLOAD_VERSION 1u

/* ------------------------------------------------------------------------
 * Payload: one worker's compressed bucket, one contiguous buffer, every
 * section 16-byte aligned:
 *   header (64 B) | idx: u32[k] strictly ascending | val: i8[k], f16[k] or
 *   f32[k] | scale: f32[nblocks] (int8 only; block b covers payload entries
 *   [b*1024, (b+1)*1024))
 * The paper leaves the layout of Com_grads open (Alg. 2 names only
 * top_k(grads, ratio)); this one is defined here.
 * ---------------------------------------------------------------------- */
typedef struct nsml_payload_header {
  uint32_t magic;     /* NSML_PAYLOAD_MAGIC */
  uint32_t version;   /* NSML_PAYLOAD_VERSION */
  uint64_t n;         /* elements in the dense bucket */
  uint64_t k;         /* survivors = ceil(ratio*n) */
  uint32_t bits;      /* NSML_BITS_INT8, NSML_BITS_FP16 or NSML_BITS_FP32 */
  uint32_t qblock;    /* NSML_QBLOCK */
  uint64_t nblocks;   /* ceil(k/qblock) for int8, else 0 */
  uint64_t idx_off;   /* byte offsets from the start of the payload */
  uint64_t val_off;
  uint64_t scale_off; /* int8 only, else 0 */
} nsml_payload_header;

/* ------------------------------------------------------------------------
 * Host controller -- Alg. 1, Eq. 1-3.
 * ---------------------------------------------------------------------- */
typedef struct nsml_ctrl nsml_ctrl; /* opaque, host memory, owned by the library */

typedef struct nsml_ctrl_params {
  double ratio_init;     /* 0.01  Alg. 1 Step 1 */
  double ratio_min;      /* 0.005 Eq. 3 */
  double ratio_max;      /* 1.0   Eq. 3 */
  double alpha;          /* 0.5   Section 4.1 */
  double beta1;          /* start-up increment; not given in the paper: 0.1 */
  double beta2;          /* 0.01  Section 4.1 */
  double bdp_frac;       /* 0.9   Eq. 3 */
  double rtt_excess;     /* start-up ends when a transfer time exceeds
                            rtt_excess*RTprop; not given in the paper: 1.25 */
  int32_t startup_max_steps; /* not given ("first few steps"): 10; 0 = no start-up */
  int32_t btlbw_window;  /* samples the BtlBw maximum runs over: 10; 0 = all-time
                            (the literal reading of Alg. 1) */
  int32_t rtprop_window; /* samples the RTprop minimum runs over: 100; 0 = all-time */
  int32_t reserved;
} nsml_ctrl_params;

typedef struct nsml_ctrl_state {
  double ratio;   /* ratio the last call returned */
  double ebb;     /* Eq. 1 of the last sample, bytes/s */
  double btlbw;   /* bytes/s */
  double rtprop;  /* seconds (+inf before the first sample) */
  double bdp;     /* Eq. 2, bytes */
  int32_t phase;  /* 0 = start-up, 1 = NetSense */
  int32_t startup_steps;
  int64_t calls;
} nsml_ctrl_state;

/* Fills *p with the defaults listed above.  Returns NSML_ERR_ARG if p is NULL. */
int nsml_ctrl_default_params(nsml_ctrl_params* p);

/* Creates a controller.  p == NULL takes the defaults.  Parameters are checked
 * (0 < ratio_min <= ratio_init <= ratio_max <= 1, 0 < alpha < 1, beta1, beta2 > 0,
 * bdp_frac > 0, rtt_excess >= 1, windows and steps >= 0; windows <= 4096):
 * NSML_ERR_ARG otherwise.  *out is written only on success; free it with
 * nsml_ctrl_destroy (NULL is allowed there). */
int nsml_ctrl_create(const nsml_ctrl_params* p, nsml_ctrl** out);
void nsml_ctrl_destroy(nsml_ctrl* c);

/* Alg. 1, one call per gradient-transmission interval i.
 *   last_bytes, last_seconds  size and measured transfer time of interval i-1
 *                             (ignored on the first call: nothing was sent yet)
 *   next_dense_bytes          size the upcoming transfer would have at ratio 1;
 *                             Eq. 3 compares ratio*next_dense_bytes with
 *                             bdp_frac*BDP
 *   ratio_out                 host pointer, receives the ratio for interval i
 * First call: returns ratio_init.  Start-up calls add beta1 until a transfer
 * time exceeds rtt_excess*RTprop, startup_max_steps increments were made or the
 * ratio reached ratio_max; the call that ends start-up, and every later call,
 * applies Eq. 1-3: EBB = last_bytes/last_seconds, BtlBw = max EBB, RTprop = min
 * transfer time, BDP = BtlBw*RTprop, then ratio = max(ratio_min, ratio*alpha) if
 * ratio*next_dense_bytes > bdp_frac*BDP else min(ratio_max, ratio+beta2).
 * All arithmetic is IEEE double in the operand order written here.
 * Errors: NSML_ERR_ARG for NULL pointers, last_seconds <= 0 or non-finite,
 * negative or non-finite sizes; the state is then unchanged. */
int nsml_select_ratio(nsml_ctrl* c, double last_bytes, double last_seconds,
                      double next_dense_bytes, double* ratio_out);

/* Copies the controller's current estimates to *out (host pointer). */
int nsml_ctrl_get_state(const nsml_ctrl* c, nsml_ctrl_state* out);

/* Checkpointing: the state is a flat blob of nsml_ctrl_save_bytes() bytes.
 * nsml_ctrl_save writes it to buf (capacity cap, NSML_ERR_CAPACITY if too
 * small); nsml_ctrl_load replaces c's parameters and state from such a blob
 * (NSML_ERR_ARG if the blob's size or tag is wrong; c is then unchanged). */
size_t nsml_ctrl_save_bytes(const nsml_ctrl* c);
int nsml_ctrl_save(const nsml_ctrl* c, void* buf, size_t cap);
int nsml_ctrl_load(nsml_ctrl* c, const void* buf, size_t bytes);

/* ------------------------------------------------------------------------
 * Sizes (pure host arithmetic; 0 is returned for arguments out of range).
 * ---------------------------------------------------------------------- */
/* k = ceil(ratio*n) evaluated in IEEE double, clamped to [1, n] (Alg. 2 Step 3
 * gives only top_k(grads, ratio); ceil is the reading used). */
int64_t nsml_k_of(int64_t n, double ratio);
/* Exact size in bytes of the payload nsml_compress writes for (n, ratio, bits). */
size_t nsml_payload_bytes(int64_t n, double ratio, int bits);
/* Scratch needed by nsml_compress for a bucket of n elements (any ratio, bits). */
size_t nsml_workspace_bytes(int64_t n, int grad_dtype);
/* Scratch needed by nsml_decompress_accumulate for (n, W). */
size_t nsml_accumulate_workspace_bytes(int64_t n, int W);

/* ------------------------------------------------------------------------
 * nsml_compress -- Alg. 2 Steps 2-3 and the value codec, one flat bucket.
 *
 *   grad        device pointer, 16-byte aligned: n elements, float32
 *               (NSML_F32) or bfloat16 (NSML_BF16, widened exactly to float32).
 *               Values must be finite.
 *   n           1 .. NSML_MAX_N
 *   ratio       kept fraction in (0, 1]; k = nsml_k_of(n, ratio)
 *   bits        NSML_BITS_INT8: per block of 1024 consecutive survivors
 *               scale = maxabs/127, code = clamp(rint(v/scale), +-127), both
 *               IEEE float32 divisions, round half to even, denormals kept;
 *               scale 0 gives codes 0.  (Not in the paper.)
 *               NSML_BITS_FP16: float32 -> binary16, round to nearest even
 *               (Alg. 2 Step 1 "quantize"); |v| >= 65520 saturates to +-65504.
 *               NSML_BITS_FP32: the survivors' float32 values as they are
 *               (Alg. 2 when Step 1 does not quantise).
 *   prune_mask  device pointer (4-byte aligned) to ceil(n/32) words, bit (i&31)
 *               of word i>>5 set = parameter i is pruned: its gradient counts as
 *               +0.0 (Alg. 2 Step 2).  NULL = nothing pruned.
 *   payload     device pointer, 16-byte aligned, capacity payload_capacity >=
 *               nsml_payload_bytes(n, ratio, bits) (else NSML_ERR_CAPACITY)
 *   workspace   device pointer, 256-byte aligned, workspace_bytes >=
 *               nsml_workspace_bytes(n, grad_dtype)
 *
 * Result: the k entries of largest magnitude (compared on the float32 bit
 * pattern with the sign cleared; ties: larger magnitude first, then lower
 * index), in ascending index order; exactly k entries even if fewer than k
 * gradients are non-zero.  The result is unique, so the payload is
 * bit-reproducible.  Device-detected: NSML_ERR_NONFINITE (payload contents
 * then unspecified), NSML_ERR_TIMEOUT.
 * ---------------------------------------------------------------------- */
int nsml_compress(const void* grad, int64_t n, int grad_dtype, double ratio, int bits,
                  const uint32_t* prune_mask, void* payload, size_t payload_capacity,
                  void* workspace, size_t workspace_bytes, void* stream);

/* Which of its two internal strategies nsml_compress takes for (n, ratio) on
 * the current device.  Both give the same payload; this is information for
 * byte accounting (the paper prescribes no strategy).
 *   NSML_STRATEGY_LIST   a stratified sample bounds the threshold from below,
 *                        one streaming pass keeps the candidates above the
 *                        bound, an exact radix select runs on that list
 *   NSML_STRATEGY_DENSE  the radix select runs over the bucket itself (high
 *                        kept fractions, and buckets too small to sample)
 * Returns the strategy, or NSML_ERR_ARG / NSML_ERR_CUDA. */
#define NSML_STRATEGY_LIST 0
#define NSML_STRATEGY_DENSE 1
int nsml_compress_strategy(int64_t n, double ratio);

/* nsml_set_list_block_candidates -- a tuning knob of the list strategy, for the
 * whole process: about how many candidates one thread block of the list stage
 * takes when the list is short (up to about a million candidates).  The result
 * of nsml_compress does not depend on it.  Fewer candidates per block = more
 * blocks = a shorter list stage for a call that has the GPU to itself; more
 * candidates per block = fewer SMs held while the stage waits for memory, which
 * is what counts when several buckets are compressed on several streams at
 * once.  Above the default the gather kernel in front of the list stage also
 * runs as one block per group of segments instead of two, and long lists get
 * one list-stage block per SM instead of two.  Measured on one
 * B200, 25M-element buckets, ratio 0.01, int8: 2048 -> a lone call 65 us;
 * 4096 -> 68 us, the eight-stream step of 20 calls and 5 sums 0.70 ms;
 * 8192 -> 81 us and 0.63 ms.
 *   candidates   1024 ... 8192; the default is 4096
 * Returns NSML_OK, or NSML_ERR_ARG for a value out of range (nothing changes).
 * Takes effect for calls made after it returns. */
int nsml_set_list_block_candidates(int candidates);

/* ------------------------------------------------------------------------
 * nsml_decompress_accumulate -- dense += sum over W payloads (plain sum, no
 * averaging), after optionally zeroing dense.
 *
 *   payloads    HOST array of W device pointers (16-byte aligned), each a payload
 *               written by nsml_compress (or laid out the same way) for this n;
 *               payloads of different codecs may be mixed; 1 <= W <= NSML_MAX_WORKERS
 *   dense       device pointer, 16-byte aligned, n float32; read unless
 *               zero_first, always written
 *   zero_first  non-zero: dense is overwritten by the sum; zero: the sum is
 *               added to what dense holds
 *   workspace   device pointer, 256-byte aligned, >=
 *               nsml_accumulate_workspace_bytes(n, W)
 *
 * Values are dequantised as float(code)*scale (one float32 multiply),
 * float(half) or taken as they are, and added in float32 in worker order w = 0..W-1, each dense
 * element by one thread: the result is deterministic.  Device-detected:
 * NSML_ERR_PAYLOAD if a header does not match (magic, version, n, bits, k) or
 * an index is >= n; nothing is written out of range.  A header is trusted as
 * to how long the payload is: a caller that receives payloads from other
 * workers and knows how many bytes arrived should use the _sized variant.
 * ---------------------------------------------------------------------- */
int nsml_decompress_accumulate(const void* const* payloads, int W, float* dense, int64_t n,
                               int zero_first, void* workspace, size_t workspace_bytes,
                               void* stream);

/* The same sum (Section 4.2 Step 3, AllGather pattern of Section 5.3) for
 * payloads whose buffer sizes are known: payload_bytes is a HOST array of W
 * sizes in bytes (each >= 64, else NSML_ERR_ARG).  A payload whose header
 * describes more bytes than its buffer holds (a truncated transfer, a k field
 * corrupted upwards) is reported as NSML_ERR_PAYLOAD on the device and none of
 * its entries is read. */
int nsml_decompress_accumulate_sized(const void* const* payloads, const size_t* payload_bytes, int W,
                                     float* dense, int64_t n, int zero_first, void* workspace,
                                     size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------
 * nsml_decompress_accumulate_static -- the same sum as
 * nsml_decompress_accumulate, for callers that have no device scratch to give
 * and no way to get any: code that runs where cudaMalloc must not be called
 * (inside a region that forbids allocation, a plug-in whose host owns every
 * byte of device memory, an error path after the allocator has failed).  The
 * paper has no counterpart; this is a convenience of the library.
 *
 * The scratch (block offsets and the status word) lives in one array of
 * NSML_STATIC_SCRATCH_BYTES bytes that is part of the library image: every GPU
 * that loads the library holds it until the process exits.  In exchange the
 * call is limited to n <= NSML_STATIC_MAX_N and W <= NSML_STATIC_MAX_WORKERS;
 * larger arguments are refused with NSML_ERR_CAPACITY and nothing is enqueued.
 * The call, and everything it calls, allocates no host or device memory (its
 * launches are never bracketed by the events of nsml_prof_enable, which would
 * allocate, so they do not show in nsml_prof_read).
 *
 *   payloads, W, dense, n, zero_first, stream   as for nsml_decompress_accumulate
 *   status_out  host pointer or NULL.  NULL: the call returns after enqueueing.
 *               Non-NULL: the call also synchronises `stream` and stores the
 *               device-detected status (NSML_OK or NSML_ERR_PAYLOAD) there.
 *               The caller never sees the scratch, so the asynchronous form
 *               (NULL) cannot report a device-detected error afterwards.
 *
 * The first call on each device looks up the array's device address (once per
 * device, with that device current); make that first call outside any stream
 * capture.  All calls on a device share the one array and it keeps what the
 * last call left in it: the status word is cleared at the start of each call,
 * and two calls whose device work overlaps (different streams, or a second
 * call before the first finished on another stream) race on it -- serialise
 * them.  Results are bit-identical to nsml_decompress_accumulate.
 * ---------------------------------------------------------------------- */
#define NSML_STATIC_MAX_N 16777216LL /* 2^24 elements (64 MiB of float32) */
#define NSML_STATIC_MAX_WORKERS 8
#define NSML_STATIC_SCRATCH_BYTES 66048 /* 256 + 8 * (2^24 / 8192 + 1) * 4, rounded up to 256 */
int nsml_decompress_accumulate_static(const void* const* payloads, int W, float* dense, int64_t n,
                                      int zero_first, void* stream, int* status_out);

/* ------------------------------------------------------------------------
 * The rest of Alg. 2 around the top-k step.
 * ---------------------------------------------------------------------- */

/* nsml_grad_l2 -- the L2 norm of Alg. 2 Step 1 ("calculate_L2_norm(grads)"):
 * sqrt(sum g_i^2), every square and the sum in float64.
 *   grad, n, grad_dtype   as for nsml_compress (no pruning mask: Step 1 comes
 *                         before Step 2)
 *   workspace   device pointer, 256-byte aligned, >= nsml_l2_workspace_bytes()
 *   l2_out      host pointer or NULL.  NULL: the call returns after enqueueing
 *               and the sum of squares (float64) is left at byte offset 8 of
 *               `workspace`.  Non-NULL: the call synchronises `stream` and
 *               stores the norm there.
 * The adds follow a fixed order for a given device, so the value is
 * reproducible run to run.  NSML_ERR_NONFINITE if the bucket holds NaN or Inf
 * (returned when l2_out is given, else left in the status word). */
size_t nsml_l2_workspace_bytes(void);
int nsml_grad_l2(const void* grad, int64_t n, int grad_dtype, void* workspace, size_t workspace_bytes,
                 void* stream, double* l2_out);

/* nsml_quantize_gate -- the decision of Alg. 2 Step 1, host arithmetic only:
 * if ratio < tr_q and l2 > tr_d the values are sent as 16-bit floats and the
 * ratio is doubled (capped at 1; the paper states no cap), else the values are
 * sent with `plain_bits` (NSML_BITS_FP32 is the paper's case) at the ratio
 * given.  tr_q ("quantization check threshold") and tr_d ("gradient density
 * threshold") are inputs of Alg. 2; the paper gives no values for them.
 * NSML_ERR_ARG for NULL outputs, a ratio outside (0, 1], NaN thresholds or a
 * negative norm. */
int nsml_quantize_gate(double ratio, double l2, double tr_q, double tr_d, int plain_bits,
                       double* ratio_out, int* bits_out);

/* Alg. 2 Step 2: pruning_rate = 0.5 * (1 - ratio).  The number of parameters
 * that rate stands for is read as m = ceil(pruning_rate * n) in IEEE double
 * (0 for arguments out of range). */
int64_t nsml_pruned_count(int64_t n, double ratio);
size_t nsml_prune_workspace_bytes(int64_t n);

/* nsml_prune_mask_build -- Alg. 2 Step 2 ("prune_weights(pruning_rate)"): marks
 * the m = nsml_pruned_count(n, ratio) parameters of smallest magnitude
 * (compared on the float32 bit pattern with the sign cleared; ties: smaller
 * magnitude first, then lower index -- the paper states no tie rule).
 *   weights     device pointer, 16-byte aligned, n finite float32
 *   prune_mask  device pointer (4-byte aligned), ceil(n/32) words, written in
 *               the layout nsml_compress reads; bits past n are 0
 *   workspace   device pointer, 256-byte aligned, >= nsml_prune_workspace_bytes(n)
 * Nothing is remembered between calls: the mask is rebuilt from the weights
 * every time (pruned parameters "are not permanently removed").
 * Device-detected: NSML_ERR_NONFINITE. */
int nsml_prune_mask_build(const float* weights, int64_t n, double ratio, uint32_t* prune_mask,
                          void* workspace, size_t workspace_bytes, void* stream);

/* nsml_compress_feedback -- nsml_compress with the local accumulation of the
 * gradients that sparsification filters out (Section 4.2 Step 3: "accumulate
 * the local filtered gradients for further aggregation and transmission"),
 * read as a residual kept by the caller between steps:
 *   acc      = grad + residual          (one float32 add per element)
 *   payload  = nsml_compress(acc, ratio, bits, prune_mask)
 *   residual = acc, and at every selected index i: acc[i] - v'_i, v' being the
 *              value nsml_decompress_accumulate reconstructs (one float32
 *              subtraction), so that the quantisation error is carried too
 *   residual    device pointer, 16-byte aligned, n float32, read and written;
 *               zero it before the first step
 *   all other arguments as for nsml_compress (workspace of
 *   nsml_workspace_bytes(n, NSML_F32) bytes).
 * A pruned parameter is not sent but keeps accumulating in the residual. */
int nsml_compress_feedback(const void* grad, float* residual, int64_t n, int grad_dtype, double ratio,
                           int bits, const uint32_t* prune_mask, void* payload, size_t payload_capacity,
                           void* workspace, size_t workspace_bytes, void* stream);

/* nsml_compress_adaptive -- Alg. 2 as a whole, in its order:
 *   Step 1  if ratio < tr_q: L2 norm (device), gate (host; the call waits for
 *           the norm, so it synchronises `stream` once in that case)
 *   Step 2  if weights != NULL: prune_mask is rebuilt from them at the ratio
 *           Step 1 left (prune_mask must then be writable, ceil(n/32) words);
 *           if weights == NULL: prune_mask is used as given (may be NULL)
 *   Step 3  nsml_compress at that ratio and codec
 *   payload_capacity >= nsml_adaptive_payload_bytes(n, ratio, tr_q, plain_bits)
 *   (the larger of the two outcomes); workspace >=
 *   nsml_adaptive_workspace_bytes(n, grad_dtype)
 *   ratio_used, bits_used   host pointers, receive what Steps 2-3 used
 *   l2_out      host pointer or NULL: the norm, or -1 when it was not needed
 * Selection is on the float32 magnitudes and only the survivors are converted
 * to 16 bits (Alg. 2 converts before selecting; the survivors differ only
 * where the conversion creates ties). */
size_t nsml_adaptive_payload_bytes(int64_t n, double ratio, double tr_q, int plain_bits);
size_t nsml_adaptive_workspace_bytes(int64_t n, int grad_dtype);
int nsml_compress_adaptive(const void* grad, int64_t n, int grad_dtype, double ratio, double tr_q,
                           double tr_d, int plain_bits, const float* weights, uint32_t* prune_mask,
                           void* payload, size_t payload_capacity, void* workspace,
                           size_t workspace_bytes, void* stream, double* ratio_used, int* bits_used,
                           double* l2_out);

/* Host-buffer variants: the same operations for callers whose gradients and
 * payloads live in host memory (pinned memory gives asynchronous copies).
 * `device_scratch` (device pointer, 256-byte aligned) must hold
 * nsml_compress_host_scratch_bytes(n, grad_dtype, ratio, bits), respectively
 * nsml_accumulate_host_scratch_bytes(n, W, total_payload_bytes); the call copies
 * the inputs to the device, runs the operation and copies the result back, all
 * on `stream`, and returns without synchronising.  payload_host / dense_host
 * are valid once the stream has been synchronised.
 * The payloads handed to nsml_decompress_accumulate_host may themselves be the
 * output of an earlier asynchronous call on the same stream, so their headers
 * are checked on the device, against payload_bytes[w]: a payload that does not
 * match n, or that describes more bytes than were handed over, is reported as
 * NSML_ERR_PAYLOAD in the status word and none of its entries is read. */
size_t nsml_compress_host_scratch_bytes(int64_t n, int grad_dtype, double ratio, int bits);
int nsml_compress_host(const void* grad_host, int64_t n, int grad_dtype, double ratio, int bits,
                       const uint32_t* prune_mask_host, void* payload_host,
                       size_t payload_capacity, void* device_scratch, size_t scratch_bytes,
                       void* stream);
size_t nsml_accumulate_host_scratch_bytes(int64_t n, int W, size_t total_payload_bytes);
int nsml_decompress_accumulate_host(const void* const* payloads_host, const size_t* payload_bytes,
                                    int W, float* dense_host, int64_t n, int zero_first,
                                    void* device_scratch, size_t scratch_bytes, void* stream);

/* Synchronises `stream`, then copies the status word of `workspace` (or of a
 * host-variant `device_scratch`) to *status_out (host pointer): NSML_OK or the
 * first device-detected error of the last call that used it. */
int nsml_last_status(const void* workspace, void* stream, int* status_out);

/* Self-test of the bounded waits between thread blocks (the cooperative
 * kernels of Alg. 2 Step 3 meet at barriers in global memory; every such wait
 * gives up after a fixed number of polls instead of hanging).  Enqueues a
 * two-block kernel whose barrier target can never be reached, with a wait
 * limit of max_polls polls (1 .. 65536; a fraction of a millisecond to a few
 * milliseconds): each block gives up, the kernel returns by itself and the
 * status word of `workspace` (device pointer, 256-byte aligned, >= 256 bytes;
 * any compress workspace will do) reads NSML_ERR_TIMEOUT afterwards.  The
 * workspace stays usable: every call clears its control block first. */
int nsml_selftest_bounded_wait(void* workspace, size_t workspace_bytes, int max_polls, void* stream);

/* Static, NUL-terminated description of a status code. */
const char* nsml_strerror(int status);

/* ------------------------------------------------------------------------
 * Instrumentation (optional; off by default).
 * ---------------------------------------------------------------------- */
/* Number of distinct kernels the library launches, and their names. */
int nsml_kernel_count(void);
const char* nsml_kernel_name(int kernel_id);
/* Total kernel launches made by this process through the library so far. */
int64_t nsml_launch_count(void);
/* on != 0: bracket every kernel launch with CUDA events on its stream, so that
 * per-kernel device time can be read back; slows the host side slightly.
 * Turning it off drops recorded samples. */
int nsml_prof_enable(int on);
/* Synchronises the recorded events and returns, for kernel_id, the summed
 * device time in milliseconds and the number of launches since the last reset. */
int nsml_prof_read(int kernel_id, double* total_ms, int64_t* launches);
int nsml_prof_reset(void);

#ifdef __cplusplus
}
#endif
#endif /* NSML_H */
