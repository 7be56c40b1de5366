/*
 * tsq — threshold splitting (TS) + token-wise adaptive bit quantisation (TAB-Q) of an LLM
 * split-point hidden state, on one NVIDIA B200 (sm_100a).
 *
 * Method: "Memory- and Latency-Constrained Inference of Large Language Models via Adaptive
 * Split Computing", Sec. II-C.  Encode = Eq. "ts" (outliers with |x| >= tau leave, undistorted,
 * as a CSR list) followed, per token row, by Algorithm 1 (TAB-Q) built on Eq. "Proposed" (AIQ):
 * a per-token min/max range over the magnitudes, a per-token bit-width chosen from a candidate
 * list by the distortion test, and the codes packed into word-aligned bit-planes.  Decode =
 * Eq. "dequnt": unpack, (code + zero-point) * scale, outliers written back.
 *
 * Conventions for every call:
 *  - plain C ABI; every pointer is marked HOST or DEVICE; the caller owns every buffer;
 *  - tsq_encode / tsq_decode only enqueue work on `cuda_stream` (a cudaStream_t passed as
 *    void*, NULL = the default stream): they never synchronise, allocate or copy to the host;
 *  - errors are return values.  Conditions that only the GPU can see (outlier capacity
 *    exceeded, malformed blob, a bounded wait that ran out) are recorded in the blob header's
 *    `status` (encode) and in the workspace (encode and decode) and are read with
 *    tsq_blob_info / tsq_workspace_status;
 *  - device tensors are contiguous row-major [tokens x hidden], 16-bit elements, base address
 *    16-byte aligned;
 *  - arithmetic is IEEE binary32, round-to-nearest-even, true division semantics, no
 *    flush-to-zero: results are bit-identical to a scalar evaluation of the paper's formulas.
 */
#ifndef TSQ_H_
#define TSQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct tsq_plan tsq_plan_t; /* opaque; host-owned; immutable after creation; may be shared by threads */

typedef enum {
  TSQ_OK = 0,
  TSQ_ERR_INVALID_ARG = 1,
  TSQ_ERR_UNSUPPORTED = 2,      /* legal for the method, declined by the GPU path (e.g. hidden % 8 != 0) */
  TSQ_ERR_BUFFER_TOO_SMALL = 3,
  TSQ_ERR_CUDA = 4,             /* a CUDA runtime call failed */
  TSQ_ERR_CORRUPT_BLOB = 5,
  TSQ_ERR_OUTLIER_OVERFLOW = 6, /* more outliers than the plan's capacity; the excess was dropped */
  TSQ_ERR_TIMEOUT = 7           /* a bounded device-side wait ran out; re-initialise the workspace */
} tsq_status_t;

typedef enum { TSQ_F16 = 0, TSQ_BF16 = 1 } tsq_dtype_t;

/*
 * Which values Eq. "Proposed" quantises.
 *   TSQ_VARIANT_MAGNITUDES     Algorithm 1 as printed: sign and magnitude are separated first, a b-bit level is
 *                              one sign bit + a (b-1)-bit code of the magnitude, Q_max = 2^(b-1) - 1.
 *   TSQ_VARIANT_SIGNED_VALUES  Eq. "Proposed" applied to the signed inliers themselves (the other reading of
 *                              Sec. II-C.2, without Algorithm 1's first two steps): min and max are those of
 *                              the signed values of T_below (outlier slots count as +0), a b-bit level is a
 *                              b-bit code, Q_max = 2^b - 1, the zero-point may be negative, no sign plane.
 * A blob records its variant (header byte bits[7]) and is decoded only by a plan of the same variant.
 */
#define TSQ_VARIANT_MAGNITUDES 0
#define TSQ_VARIANT_SIGNED_VALUES 1

typedef struct {
  size_t blob_bytes;      /* bytes of the blob buffer for `tokens` rows (capacity, not payload) */
  size_t workspace_bytes; /* bytes of the workspace the plan needs (independent of `tokens`) */
} tsq_sizes_t;

typedef struct {
  uint32_t status;        /* tsq_status_t recorded by the encoder */
  uint32_t tokens, hidden, dtype;
  uint64_t total_words;   /* 32-bit words of bit-planes in use */
  uint64_t total_outliers;
  uint64_t payload_bytes; /* bytes a sender would transmit: header + per-token fields + planes + CSR */
} tsq_info_t;

/*
 * Blob format "TSQ1" (little endian; every section starts on a 16-byte boundary; capacities are
 * those of the call's `tokens` and the plan; only the first total_words / total_outliers entries
 * of the last two sections are meaningful).  WPP = ceil(hidden / 32).
 *
 *   header   64 B  u32 magic 'TSQ1' | u32 version=1 | u32 dtype | u32 hidden | u32 tokens |
 *                  u32 n_bits | u8 bits[7] | u8 variant | f32 tau | f32 delta | u64 total_words |
 *                  u64 total_outliers | u32 status | u32 outlier_capacity
 *   bits     u8  [tokens]      chosen bit-width b* (1 sign bit + (b*-1)-bit magnitude code; signed-values
 *                              variant: a b*-bit code)
 *   scale    f32 [tokens]      AIQ scale s
 *   zp       i32 [tokens]      AIQ zero-point, restore = (code + zp) * s.  The decoder accepts 0 <= zp < 2^22
 *                              (|zp| < 2^22 in the signed-values variant) and reports any other value as
 *                              TSQ_ERR_CORRUPT_BLOB: 16-bit inputs cannot produce more (the minimum over
 *                              the scale is at most 2^11 Q_max, below 2^19), and the bound keeps code + zp
 *                              exact in binary32
 *   word_off u32 [tokens+1]    exclusive prefix sum of b* x WPP
 *   out_ptr  u32 [tokens+1]    CSR row pointers (exclusive prefix sum of per-token outlier counts)
 *   words    u32 [tokens x bmax x WPP]  token t owns b* x WPP words from word_off[t], interleaved
 *                  per group of 32 elements: word g*b* + k is plane k of elements 32g .. 32g+31,
 *                  plane 0 = sign bits of the inliers, plane 1+k = bit k of the magnitude codes;
 *                  bit i of a group's word belongs to element 32g + i; pad bits are 0.  Signed-values
 *                  variant: plane k = bit k of the code, no sign plane
 *   outl     u32 [outlier_capacity]     (column << 16) | original 16-bit pattern, columns ascending
 */

/*
 * Create a plan: parameters of TS (tau, Eq. "ts") and of TAB-Q (candidate bit-widths and the
 * distortion tolerance delta of Algorithm 1; the paper's default is delta = 0.2).
 *   out          HOST   receives the plan; destroy with tsq_plan_destroy
 *   device              CUDA device ordinal the plan's kernels will run on
 *   hidden              row length H, 8 <= H <= 65536, H % 8 == 0 (else TSQ_ERR_UNSUPPORTED)
 *   max_tokens          largest `tokens` any call will pass (>= 0); tokens * H < 2^32 and
 *                       tokens * bmax * WPP < 2^32
 *   tau                 threshold; |x| >= tau, NaN and +-Inf become outliers.  +INF disables TS
 *                       for finite values, tau <= 0 makes every element an outlier.  NaN is invalid
 *   bits         HOST   n_bits strictly increasing candidates, each in [2, 8]; 1 <= n_bits <= 7
 *   delta               tolerance on the mean absolute code distortion (may be negative: no
 *                       lower candidate is ever accepted)
 *   max_outliers        CSR capacity in entries; 0 = worst case tokens * H
 * Queries device attributes; allocates no device memory.
 */
tsq_status_t tsq_plan(tsq_plan_t **out, int device, tsq_dtype_t dtype, int32_t hidden, int64_t max_tokens,
                      float tau, const int32_t *bits, int32_t n_bits, float delta, int64_t max_outliers);

/*
 * The same with the variant chosen (TSQ_VARIANT_*; tsq_plan is this call with TSQ_VARIANT_MAGNITUDES).  Any other
 * value is TSQ_ERR_INVALID_ARG.  Every other call takes plans of either variant.
 */
tsq_status_t tsq_plan_variant(tsq_plan_t **out, int device, tsq_dtype_t dtype, int32_t hidden, int64_t max_tokens,
                              float tau, const int32_t *bits, int32_t n_bits, float delta, int64_t max_outliers,
                              int32_t variant);

/* Buffer sizes for a call with `tokens` rows (0 <= tokens <= max_tokens). `out` is HOST. */
tsq_status_t tsq_plan_sizes(const tsq_plan_t *plan, int64_t tokens, tsq_sizes_t *out);

/*
 * Zero a workspace (DEVICE, workspace_bytes, 16-byte aligned) on `cuda_stream`.  Required once
 * before the buffer's first use and after any TSQ_ERR_TIMEOUT; encode and decode leave it ready
 * for the next call.  One workspace serves one call at a time: calls that may overlap on the GPU
 * need separate workspaces.  (Variable-length placement, the prefix sums behind word_off and
 * out_ptr, is resolved inside the encode kernel through this buffer.)
 */
tsq_status_t tsq_workspace_init(const tsq_plan_t *plan, void *ws_dev, size_t ws_bytes, void *cuda_stream);

/*
 * Set how long the encoder's device-side waits may last before they give up with TSQ_ERR_TIMEOUT.  The
 * only such wait is the placement look-back: a row's offsets are the prefix sums over every earlier
 * row, and a row polls the workspace until those rows have published theirs.  `polls` counts polls of
 * one descriptor (200 ns apart for the first 32, then 1 us apart); 0 restores the built-in limit of
 * 2^20 polls (about one second), which is also what tsq_workspace_init sets.  A wait can only run out
 * when the workspace was not initialised, is shared by calls that overlap on the GPU, or was
 * overwritten: the limit exists so that such a mistake ends in a status instead of a hang.  The
 * setting is kept in the workspace (DEVICE) and is written on `cuda_stream`.
 */
tsq_status_t tsq_workspace_set_wait_limit(void *ws_dev, uint32_t polls, void *cuda_stream);

/*
 * Encode x (DEVICE, [tokens x hidden]) into blob (DEVICE, >= blob_bytes from tsq_plan_sizes,
 * 16-byte aligned): TS (Eq. "ts") + TAB-Q (Algorithm 1, token-wise) + bit-plane packing, one
 * kernel launch.  tokens == 0 writes an empty, valid blob.  Returns argument errors before
 * anything is enqueued.
 */
tsq_status_t tsq_encode(const tsq_plan_t *plan, const void *x_dev, int64_t tokens, void *blob_dev,
                        size_t blob_bytes, void *ws_dev, size_t ws_bytes, void *cuda_stream);

/*
 * The same encode as tsq_encode, for callers that cannot give it a workspace.  (The paper has no
 * counterpart: this is a convenience of the library.)  Some hosts of this codec are not allowed to
 * allocate device memory where they call it: code running inside a region that forbids allocation
 * (a latency-critical serving loop with a frozen memory pool, a plug-in whose embedding runtime owns
 * all device memory, a thread that must never take the allocator's lock).  For them the look-back
 * scratch lives in a fixed array inside the library image instead of in a caller-allocated workspace;
 * x_dev and blob_dev are still the caller's.
 *   - Limit: the plan's max_tokens must be <= 16384 (the array is 256 KiB + 256 B per device, held
 *     by every device that loads the library until the process exits); larger plans are refused with
 *     TSQ_ERR_UNSUPPORTED before anything is enqueued.
 *   - The call allocates and frees nothing.  The first call on a device looks up the array's device
 *     address (a one-time host-side query with that device made current for a moment); make that
 *     first call before any stream capture begins.
 *   - Each call first clears the part of the array it uses, on `cuda_stream`, then encodes.  All calls
 *     on a device share the one array: two calls whose work may overlap on the GPU (different
 *     streams, no ordering between them) race on it and corrupt each other's placement.  Order them
 *     on one stream or with events.
 *   - Asynchronous conditions are reported in the blob header only (read them with tsq_blob_info).
 * Output, arguments and errors are otherwise those of tsq_encode.
 */
tsq_status_t tsq_encode_noalloc(const tsq_plan_t *plan, const void *x_dev, int64_t tokens, void *blob_dev,
                                size_t blob_bytes, void *cuda_stream);

/*
 * Decode blob (DEVICE) into y (DEVICE, [tokens x hidden]): Eq. "dequnt".  The kernel validates the
 * header against the plan and `tokens`, and every per-token field against the blob's capacities,
 * before using it; on a mismatch it writes nothing for that blob/row and records
 * TSQ_ERR_CORRUPT_BLOB (or the encoder's own non-zero status) in the workspace.
 */
tsq_status_t tsq_decode(const tsq_plan_t *plan, const void *blob_dev, size_t blob_bytes, int64_t tokens,
                        void *y_dev, void *ws_dev, size_t ws_bytes, void *cuda_stream);

/* Copy the blob's header to the host and summarise it. Synchronises `cuda_stream`. `out` is HOST. */
tsq_status_t tsq_blob_info(const void *blob_dev, tsq_info_t *out, void *cuda_stream);

/*
 * First asynchronous error recorded in the workspace since it was initialised (TSQ_OK if none),
 * for the encoder and for the decoder.  Synchronises `cuda_stream`.  Both outputs are HOST.
 */
tsq_status_t tsq_workspace_status(const void *ws_dev, uint32_t *encode_status, uint32_t *decode_status,
                                  void *cuda_stream);

/*
 * Host-buffer convenience calls (x_host / blob_host / y_host are HOST, ideally pinned; the *_dev
 * staging buffers are DEVICE and caller-owned, sized as for tsq_encode / tsq_decode).
 * tsq_encode_host copies x to the device, encodes, and copies back the header, the per-token
 * fields and only the used part of the planes and of the CSR list; *payload_bytes (HOST) receives
 * the number of meaningful bytes.  tsq_decode_host copies a blob produced that way to the device,
 * decodes and copies y back.  Both synchronise `cuda_stream` and return the asynchronous status.
 */
tsq_status_t tsq_encode_host(const tsq_plan_t *plan, const void *x_host, int64_t tokens, void *blob_host,
                             size_t blob_bytes, uint64_t *payload_bytes, void *x_dev, void *blob_dev,
                             void *ws_dev, size_t ws_bytes, void *cuda_stream);
tsq_status_t tsq_decode_host(const tsq_plan_t *plan, const void *blob_host, size_t blob_bytes, int64_t tokens,
                             void *y_host, void *blob_dev, void *y_dev, void *ws_dev, size_t ws_bytes,
                             void *cuda_stream);

/*
 * Size and latency models around the codec (host only, plain double arithmetic, no state).  They let a caller
 * take the early-exit decisions of Algorithm 2 (send the KV cache or only the hidden state, compress harder)
 * from byte counts: the model's before compression, tsq_blob_info's payload_bytes after it.  Every function
 * returns NaN for arguments outside the stated ranges.
 *
 * tsq_model_kv_bits: Eq. "bkv" (Sec. II-B), bits of KV cache held on the edge when token w (>= 1) has reached
 *   layer `layer` (1..n_layers):  2 * sum_{k<=layer} T_w Q_k + 2 * sum_{k>layer} T_{w-1} Q_k + hd * Q_layer,
 *   with T_w = w * hd and Q_k = qa_front for k < split_layer, qa_back from the split layer on (bits per element).
 * tsq_model_io_bits: Eq. "if_total", bits of the intermediate output: the whole of Eq. "bkv" when send_kv != 0,
 *   else the hidden state alone, T_w * Q_layer.
 * tsq_model_outage: P_o(R) = 1 - exp(-(2^(R/W) - 1) / gamma) (Sec. II-D.2); rate R and bandwidth W in the same
 *   unit (bits/s and Hz), gamma the received signal-to-noise ratio (linear); all three > 0.
 * tsq_model_latency: the epsilon-outage latency  bits / R * ceil(ln(epsilon) / ln(P_o(R)))  in seconds,
 *   0 < epsilon < 1 (one transmission when P_o is 0, +Inf when it is 1).
 * tsq_model_best_rate: R* = argmin over [rate_lo, rate_hi] of g(R) = ln(1 / P_o(R)) / R, by a scan of 4096
 *   cells and golden-section refinement (the paper asks for "a simple one-dimensional search").
 */
double tsq_model_kv_bits(int64_t w, int32_t layer, int32_t n_layers, int32_t split_layer, int64_t hd, double qa_front,
                         double qa_back);
double tsq_model_io_bits(int64_t w, int32_t layer, int32_t n_layers, int32_t split_layer, int64_t hd, double qa_front,
                         double qa_back, int32_t send_kv);
double tsq_model_outage(double rate, double bandwidth, double snr);
double tsq_model_latency(double bits, double rate, double bandwidth, double snr, double epsilon);
double tsq_model_best_rate(double rate_lo, double rate_hi, double bandwidth, double snr);

/* Number of kernels the library has launched in this process (all plans, all streams). */
uint64_t tsq_kernel_launch_count(void);

void tsq_plan_destroy(tsq_plan_t *plan);
const char *tsq_status_string(tsq_status_t status);

#ifdef __cplusplus
}
#endif
#endif /* TSQ_H_ */
