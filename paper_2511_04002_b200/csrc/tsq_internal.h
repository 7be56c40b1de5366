// Internal definitions shared by the host API and the kernels of the tsq library:
// blob layout ("TSQ1"), workspace control block, kernel parameter blocks.
#ifndef TSQ_INTERNAL_H_
#define TSQ_INTERNAL_H_

#include <cuda_runtime.h>
#include <stdint.h>

#include "tsq.h"

namespace tsq {

constexpr uint32_t kMagic = 0x31515354u;  // 'T','S','Q','1'
constexpr uint32_t kVersion = 1u;
constexpr int kMaxCand = 7;
constexpr int kMaxThreads = 256;          // decoder: threads per CTA, one 32-element unit per thread per pass
constexpr int kPipeMaxThreads = 320;      // pipelined encoder: compute threads (<= 256 groups) + two service warps
constexpr int kMaxDevices = 64;           // devices per process that the library keeps per-device state for
constexpr int kMaxRing = 8;               // pipelined encoder: most rows a CTA holds between packing and placement
constexpr int kEncMaxThreads = 1024;      // encoder: one CTA per row, one or two 32-element groups per thread

struct BlobHeader {
  uint32_t magic, version, dtype, hidden, tokens, n_bits;
  uint8_t bits[8];
  float tau, delta;
  unsigned long long total_words, total_outliers;
  uint32_t status, outlier_capacity;
};
static_assert(sizeof(BlobHeader) == 64, "blob header is 64 bytes");

// Byte offsets of the blob's sections for one call.
struct BlobLayout {
  unsigned long long off_bits, off_scale, off_zp, off_word_off, off_out_ptr, off_words, off_outl, total;
  unsigned long long words_capacity, outlier_capacity;
  uint32_t wpp;
};

__host__ __device__ inline unsigned long long align16(unsigned long long v) { return (v + 15ull) & ~15ull; }

// tokens * hidden < 2^32 and tokens * bmax * wpp < 2^32 are checked by the caller.
__host__ __device__ inline BlobLayout make_layout(uint32_t hidden, unsigned long long tokens, uint32_t bmax,
                                                  unsigned long long outlier_capacity) {
  BlobLayout L;
  L.wpp = (hidden + 31u) / 32u;
  L.words_capacity = tokens * bmax * L.wpp;
  L.outlier_capacity = outlier_capacity;
  unsigned long long o = 64;
  L.off_bits = o;      o = align16(o + tokens);
  L.off_scale = o;     o = align16(o + 4 * tokens);
  L.off_zp = o;        o = align16(o + 4 * tokens);
  L.off_word_off = o;  o = align16(o + 4 * (tokens + 1));
  L.off_out_ptr = o;   o = align16(o + 4 * (tokens + 1));
  L.off_words = o;     o = align16(o + 4 * L.words_capacity);
  L.off_outl = o;      o = align16(o + 4 * outlier_capacity);
  L.total = o;
  return L;
}

// Workspace: a 64-byte control block and two adjacent 64-bit descriptors per token (plane words,
// outliers).  A descriptor is (tag << 32) | value with tag = generation * 4 + flag; stale
// generations read as "not yet published", so the array never needs clearing between calls.
struct WsControl {
  uint32_t gen;          // generation of the last finished encode
  uint32_t ticket;       // next tile to hand out (self-resetting)
  uint32_t done;         // CTAs that have finished (self-resetting)
  uint32_t err;          // first error of the running encode
  uint32_t enc_status;   // first encode error since init (sticky)
  uint32_t dec_status;   // first decode error since init (sticky)
  uint32_t desc_capacity;  // tiles the descriptor array holds (set by init)
  uint32_t poll_limit;     // polls before a device-side wait gives up; 0 = the built-in limit
  uint32_t pad[8];
};
static_assert(sizeof(WsControl) == 64, "control block is 64 bytes");

constexpr uint32_t kFlagAggregate = 1, kFlagPrefix = 2, kFlagAbort = 3;
constexpr uint32_t kGenWrap = (1u << 30) - 2;

struct EncodeParams {
  const uint16_t* x;
  unsigned char* blob;
  WsControl* ws;
  unsigned long long* desc;                  // [2 * max_tokens] tile descriptors
  BlobLayout lay;
  uint32_t tokens, hidden, units, chunks;   // units = ceil(H/32), chunks = H/8
  uint32_t thr16;                            // smallest non-negative 16-bit pattern with value >= tau
  int32_t n_bits;
  int32_t bits[8];
  int32_t s_max;                             // floor(delta * H), clamped to [-1, INT32_MAX]
  uint32_t vec_store;                        // 1: every token's plane words start on a 16-byte boundary
  uint32_t direct_tiles;                     // one-CTA-per-row kernel: 1 = row index is the CTA index (every CTA resident)
  // pipelined kernel only: thread split, shared-memory strides (bytes; csr_cap in entries), ring depth in rows
  uint32_t compute_threads, park_stride, planes_stride, csr_cap, ring;
  uint32_t dtype;
  uint32_t variant;                          // 0: sign + magnitude codes; 1: codes of the signed values
  float tau, delta;
};

struct DecodeParams {
  const unsigned char* blob;
  uint16_t* y;
  WsControl* ws;
  BlobLayout lay;
  uint32_t tokens, hidden, units, chunks;
  uint32_t bmax, dtype;
  uint32_t variant;
  unsigned long long blob_bytes;
};

cudaError_t launch_encode_rows(const EncodeParams& p, int grid, int threads, int groups_per_thread, cudaStream_t stream);
cudaError_t launch_encode_pipe(const EncodeParams& p, bool full, int grid, int threads, size_t smem, cudaStream_t stream);
cudaError_t encode_pipe_attrs(bool bf16, bool full, bool signed_values, int threads, size_t smem, int* blocks_per_sm);
cudaError_t launch_decode(const DecodeParams& p, int grid, int threads, size_t smem, cudaStream_t stream);
cudaError_t decode_kernel_attrs(bool bf16, int threads, size_t smem, int* blocks_per_sm);
size_t decode_smem_bytes(uint32_t row_bytes);

}  // namespace tsq

#endif  // TSQ_INTERNAL_H_
