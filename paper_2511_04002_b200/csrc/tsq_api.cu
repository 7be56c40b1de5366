// Host side of the tsq C ABI: plan creation, buffer sizing, argument checks, launches.

#include <atomic>
#include <cmath>
#include <cstring>
#include <mutex>
#include <new>

#include "tsq_internal.h"

namespace tsq {
namespace {

std::atomic<unsigned long long> g_launches{0};

// Value of a non-negative 16-bit pattern, on the host (used once per plan, for the threshold).
float pattern_value(tsq_dtype_t dtype, uint32_t pat) {
  if (dtype == TSQ_BF16) {
    const uint32_t u = pat << 16;
    float f;
    std::memcpy(&f, &u, 4);
    return f;
  }
  const int e = (pat >> 10) & 0x1f;
  const int frac = pat & 0x3ff;
  if (e == 0x1f) return frac ? NAN : INFINITY;
  if (e == 0) return std::ldexp(static_cast<float>(frac), -24);
  return std::ldexp(static_cast<float>(frac | 0x400), e - 25);
}

// Smallest non-negative 16-bit pattern whose value is >= tau (tau is not NaN).  Patterns of
// non-negative values are ordered like the values, so a bisection over [0, +Inf pattern] finds it.
uint32_t threshold_pattern(tsq_dtype_t dtype, float tau) {
  const uint32_t inf_pat = dtype == TSQ_BF16 ? 0x7f80u : 0x7c00u;
  if (tau <= 0.0f) return 0u;
  uint32_t lo = 0u, hi = inf_pat;  // invariant: value(hi) >= tau
  while (lo < hi) {
    const uint32_t mid = (lo + hi) / 2u;
    if (pattern_value(dtype, mid) >= tau) {
      hi = mid;
    } else {
      lo = mid + 1u;
    }
  }
  return hi;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Scratch of tsq_encode_noalloc: a workspace that lives in the library image instead of in memory the
// caller allocates.  Every device that loads the library holds its own copy until the process exits.
constexpr unsigned long long kStaticMaxTokens = 16384;
constexpr size_t kStaticWsBytes = (sizeof(WsControl) + 16ull * kStaticMaxTokens + 255ull) & ~255ull;
static __device__ __align__(256) unsigned char g_static_ws[kStaticWsBytes];

// In host code `g_static_ws` is only a handle for the runtime, not an address a kernel may use: the
// device address is asked for once per device, with that device current, and kept here.
std::mutex g_static_mutex;
void* g_static_ptr[kMaxDevices] = {};

cudaError_t static_workspace(int device, void** out) {
  if (device < 0 || device >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_static_mutex);
  if (!g_static_ptr[device]) {
    int prev = 0;
    cudaError_t e = cudaGetDevice(&prev);
    if (e != cudaSuccess) return e;
    e = cudaSetDevice(device);
    if (e != cudaSuccess) return e;
    void* ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_static_ws);
    cudaSetDevice(prev);
    if (e != cudaSuccess) return e;
    if (!ptr) return cudaErrorInvalidSymbol;
    g_static_ptr[device] = ptr;
  }
  *out = g_static_ptr[device];
  return cudaSuccess;
}

__global__ void workspace_init_kernel(WsControl* ws, uint32_t desc_capacity) { ws->desc_capacity = desc_capacity; }
__global__ void workspace_wait_limit_kernel(WsControl* ws, uint32_t polls) { ws->poll_limit = polls; }

}  // namespace
}  // namespace tsq

struct tsq_plan {
  int device;
  tsq_dtype_t dtype;
  uint32_t hidden, units, chunks, row_bytes;
  unsigned long long max_tokens, max_outliers;
  float tau, delta;
  int32_t n_bits;
  int32_t bits[8];
  int32_t bmax;
  int32_t s_max;
  uint32_t thr16;
  uint32_t variant;                 // 0: sign + magnitude codes; 1: codes of the signed values
  int threads;                      // decoder CTA size, one group per thread
  int threads_half, dec_blocks_half; // the same with two groups per thread, and its resident CTAs per SM
  int enc_threads, enc_upt;         // row-at-a-time encoder: CTA size and 32-element groups per thread
  // pipelined encoder: 0 CTAs per SM when the row does not fit its shared memory
  int pipe_threads, pipe_ctas_per_sm;
  bool pipe_full;
  uint32_t pipe_compute, pipe_park, pipe_planes, pipe_csr_cap, pipe_ring;
  size_t pipe_smem;
  int sms;
  size_t dec_smem;
  size_t workspace_bytes;
};

using namespace tsq;

extern "C" {

const char* tsq_status_string(tsq_status_t status) {
  switch (status) {
    case TSQ_OK: return "ok";
    case TSQ_ERR_INVALID_ARG: return "invalid argument";
    case TSQ_ERR_UNSUPPORTED: return "unsupported by the GPU path";
    case TSQ_ERR_BUFFER_TOO_SMALL: return "buffer too small";
    case TSQ_ERR_CUDA: return "CUDA runtime error";
    case TSQ_ERR_CORRUPT_BLOB: return "corrupt blob";
    case TSQ_ERR_OUTLIER_OVERFLOW: return "outlier capacity exceeded";
    case TSQ_ERR_TIMEOUT: return "device-side wait timed out";
  }
  return "unknown status";
}

uint64_t tsq_kernel_launch_count(void) { return g_launches.load(); }

tsq_status_t tsq_plan(tsq_plan_t** out, int device, tsq_dtype_t dtype, int32_t hidden, int64_t max_tokens, float tau,
                      const int32_t* bits, int32_t n_bits, float delta, int64_t max_outliers) {
  return tsq_plan_variant(out, device, dtype, hidden, max_tokens, tau, bits, n_bits, delta, max_outliers, TSQ_VARIANT_MAGNITUDES);
}

tsq_status_t tsq_plan_variant(tsq_plan_t** out, int device, tsq_dtype_t dtype, int32_t hidden, int64_t max_tokens, float tau,
                              const int32_t* bits, int32_t n_bits, float delta, int64_t max_outliers, int32_t variant) {
  if (!out) return TSQ_ERR_INVALID_ARG;
  *out = nullptr;
  if (variant != TSQ_VARIANT_MAGNITUDES && variant != TSQ_VARIANT_SIGNED_VALUES) return TSQ_ERR_INVALID_ARG;
  if (dtype != TSQ_F16 && dtype != TSQ_BF16) return TSQ_ERR_INVALID_ARG;
  if (!bits || n_bits < 1 || n_bits > kMaxCand) return TSQ_ERR_INVALID_ARG;
  for (int i = 0; i < n_bits; ++i) {
    if (bits[i] < 2 || bits[i] > 8) return TSQ_ERR_INVALID_ARG;
    if (i > 0 && bits[i] <= bits[i - 1]) return TSQ_ERR_INVALID_ARG;
  }
  if (tau != tau || delta != delta) return TSQ_ERR_INVALID_ARG;
  if (hidden < 1 || hidden > 65536 || max_tokens < 0 || max_outliers < 0 || device < 0) return TSQ_ERR_INVALID_ARG;
  if (hidden % 8 != 0) return TSQ_ERR_UNSUPPORTED;
  const unsigned long long T = static_cast<unsigned long long>(max_tokens), H = static_cast<unsigned long long>(hidden);
  const int bmax = bits[n_bits - 1];
  const unsigned long long wpp = (H + 31) / 32;
  if (T * H >= (1ull << 32) || T * bmax * wpp >= (1ull << 32)) return TSQ_ERR_INVALID_ARG;

  tsq_plan_t* p = new (std::nothrow) tsq_plan_t();
  if (!p) return TSQ_ERR_INVALID_ARG;
  p->device = device;
  p->dtype = dtype;
  p->hidden = static_cast<uint32_t>(hidden);
  p->units = static_cast<uint32_t>(wpp);
  p->chunks = static_cast<uint32_t>(hidden / 8);
  p->row_bytes = static_cast<uint32_t>(hidden) * 2u;
  p->max_tokens = T;
  p->max_outliers = static_cast<unsigned long long>(max_outliers);
  p->tau = tau;
  p->delta = delta;
  p->n_bits = n_bits;
  for (int i = 0; i < 8; ++i) p->bits[i] = i < n_bits ? bits[i] : 0;
  p->bmax = bmax;
  p->variant = static_cast<uint32_t>(variant);
  const double smax = std::floor(static_cast<double>(delta) * static_cast<double>(hidden));
  p->s_max = smax < -1.0 ? -1 : (smax > 2147483647.0 ? 2147483647 : static_cast<int32_t>(smax));
  p->thr16 = threshold_pattern(dtype, tau);
  // decoder CTA: one 32-element group per thread, or two when the call has rows enough to fill the device
  // several times over with the smaller CTAs (a thread's fixed work, checking the header and the token's
  // fields, is then spread over 64 elements: 8 % faster at 8192 x 8192 and 32768 x 4096; with fewer rows
  // the smaller CTAs leave the device short of threads and are slower); never fewer than 64 threads while
  // the row has that many groups
  p->threads = static_cast<int>(((p->units + 31u) / 32u) * 32u);
  if (p->threads > kMaxThreads) p->threads = kMaxThreads;
  {
    const uint32_t all = static_cast<uint32_t>(p->threads), half = (((p->units + 1u) / 2u + 31u) / 32u) * 32u;
    const uint32_t floor64 = all < 64u ? all : 64u;
    p->threads_half = static_cast<int>(half > floor64 ? half : floor64);
    if (p->threads_half > p->threads) p->threads_half = p->threads;
  }
  // encoder: one thread per 32-element group, two for rows longer than kEncMaxThreads groups
  p->enc_upt = p->units > static_cast<uint32_t>(kEncMaxThreads) ? 2 : 1;
  p->enc_threads = static_cast<int>(((p->units + p->enc_upt - 1) / p->enc_upt + 31u) / 32u * 32u);
  p->dec_smem = decode_smem_bytes(p->row_bytes);
  const unsigned long long desc = T > 0 ? T : 1;
  p->workspace_bytes = static_cast<size_t>(align16(sizeof(WsControl) + 16ull * desc));

  int n_dev = 0;
  if (cudaGetDeviceCount(&n_dev) != cudaSuccess || device >= n_dev) {
    delete p;
    return TSQ_ERR_CUDA;
  }
  int prev_dev = 0;
  cudaGetDevice(&prev_dev);
  bool ok = cudaSetDevice(device) == cudaSuccess;
  int sms = 0, dec_blocks = 0;
  ok = ok && cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) == cudaSuccess;
  ok = ok && decode_kernel_attrs(dtype == TSQ_BF16, p->threads, p->dec_smem, &dec_blocks) == cudaSuccess;
  ok = ok && decode_kernel_attrs(dtype == TSQ_BF16, p->threads_half, p->dec_smem, &p->dec_blocks_half) == cudaSuccess;
  {
    // pipelined encoder: three parked rows and a ring of rows of planes and of CSR entries per CTA
    int smem_optin = 0;
    ok = ok && cudaDeviceGetAttribute(&smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device) == cudaSuccess;
    p->pipe_compute = (p->units + 31u) / 32u * 32u;
    p->pipe_full = (p->hidden % 32u == 0u) && (p->units == p->pipe_compute);  // every compute thread owns a whole group
    p->pipe_threads = static_cast<int>(p->pipe_compute) + 64;
    p->pipe_park = p->pipe_compute * 64u;
    p->pipe_planes = (static_cast<uint32_t>(p->bmax) * p->units * 4u + 127u) & ~127u;
    // A CSR list per ring slot: four entries per group (one outlier in eight elements; rows above that take
    // a slower path that holds up their CTA's placement) when that costs neither a resident CTA nor ring
    // depth below 6 (or below what two entries per group give), else two entries per group.
    p->pipe_ctas_per_sm = 0;
    p->pipe_ring = 4u;
    p->pipe_csr_cap = 2u * p->pipe_compute;
    p->pipe_smem = 0;
    int base_blocks = 0;
    uint32_t base_ring = 0;
    const bool sv = variant == TSQ_VARIANT_SIGNED_VALUES;
    for (uint32_t per_group = 2u; ok && per_group <= 4u && p->pipe_threads <= kPipeMaxThreads; per_group += 2u) {
      const uint32_t cap = per_group * p->pipe_compute;
      const auto smem_for = [&](uint32_t ring) {
        return 3u * static_cast<size_t>(p->pipe_park) + ring * (static_cast<size_t>(p->pipe_planes) + 4u * static_cast<size_t>(cap));
      };
      if (smem_for(4u) + 8192 > static_cast<size_t>(smem_optin)) break;
      int blocks = 0;
      ok = encode_pipe_attrs(dtype == TSQ_BF16, p->pipe_full, sv, p->pipe_threads, smem_for(4u), &blocks) == cudaSuccess;
      if (!ok || blocks < 1) break;
      // the deepest ring that leaves the number of resident CTAs as it is
      uint32_t ring = 4u;
      for (uint32_t r = static_cast<uint32_t>(kMaxRing); ok && r > 4u; --r) {
        if (smem_for(r) + 8192 > static_cast<size_t>(smem_optin)) continue;
        int b = 0;
        ok = encode_pipe_attrs(dtype == TSQ_BF16, p->pipe_full, sv, p->pipe_threads, smem_for(r), &b) == cudaSuccess;
        if (ok && b == blocks) {
          ring = r;
          break;
        }
      }
      if (!ok) break;
      if (per_group == 2u) {
        base_blocks = blocks;
        base_ring = ring;
      } else if (blocks != base_blocks || ring < (base_ring < 6u ? base_ring : 6u)) {
        break;  // the longer lists cost too much: keep the shorter ones
      }
      p->pipe_ctas_per_sm = blocks;
      p->pipe_ring = ring;
      p->pipe_csr_cap = cap;
      p->pipe_smem = smem_for(ring);
    }
  }
  cudaSetDevice(prev_dev);
  if (!ok || dec_blocks < 1 || sms < 1) {
    cudaGetLastError();
    delete p;
    return TSQ_ERR_CUDA;
  }
  p->sms = sms;
  *out = p;
  return TSQ_OK;
}

void tsq_plan_destroy(tsq_plan_t* plan) { delete plan; }

static BlobLayout layout_for(const tsq_plan_t* plan, unsigned long long tokens) {
  unsigned long long cap = tokens * plan->hidden;
  if (plan->max_outliers > 0 && plan->max_outliers < cap) cap = plan->max_outliers;
  return make_layout(plan->hidden, tokens, static_cast<uint32_t>(plan->bmax), cap);
}

tsq_status_t tsq_plan_sizes(const tsq_plan_t* plan, int64_t tokens, tsq_sizes_t* out) {
  if (!plan || !out || tokens < 0 || static_cast<unsigned long long>(tokens) > plan->max_tokens) return TSQ_ERR_INVALID_ARG;
  const BlobLayout L = layout_for(plan, static_cast<unsigned long long>(tokens));
  out->blob_bytes = static_cast<size_t>(L.total);
  out->workspace_bytes = plan->workspace_bytes;
  return TSQ_OK;
}

tsq_status_t tsq_workspace_init(const tsq_plan_t* plan, void* ws_dev, size_t ws_bytes, void* cuda_stream) {
  if (!plan || !ws_dev || !aligned16(ws_dev)) return TSQ_ERR_INVALID_ARG;
  if (ws_bytes < plan->workspace_bytes) return TSQ_ERR_BUFFER_TOO_SMALL;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemsetAsync(ws_dev, 0, plan->workspace_bytes, st) != cudaSuccess) return TSQ_ERR_CUDA;
  const uint32_t cap = static_cast<uint32_t>(plan->max_tokens > 0 ? plan->max_tokens : 1);
  workspace_init_kernel<<<1, 1, 0, st>>>(static_cast<WsControl*>(ws_dev), cap);
  g_launches.fetch_add(1);
  return cudaGetLastError() == cudaSuccess ? TSQ_OK : TSQ_ERR_CUDA;
}

tsq_status_t tsq_workspace_set_wait_limit(void* ws_dev, uint32_t polls, void* cuda_stream) {
  if (!ws_dev || !aligned16(ws_dev)) return TSQ_ERR_INVALID_ARG;
  workspace_wait_limit_kernel<<<1, 1, 0, static_cast<cudaStream_t>(cuda_stream)>>>(static_cast<WsControl*>(ws_dev), polls);
  g_launches.fetch_add(1);
  return cudaGetLastError() == cudaSuccess ? TSQ_OK : TSQ_ERR_CUDA;
}

// Argument checks of an encode call, made before anything is enqueued.
static tsq_status_t check_encode_args(const tsq_plan_t* plan, const void* x_dev, int64_t tokens, const void* blob_dev,
                                      size_t blob_bytes, const void* ws_dev, size_t ws_bytes) {
  if (!plan || !blob_dev || !ws_dev || tokens < 0 || static_cast<unsigned long long>(tokens) > plan->max_tokens)
    return TSQ_ERR_INVALID_ARG;
  if (tokens > 0 && !x_dev) return TSQ_ERR_INVALID_ARG;
  if (!aligned16(x_dev) || !aligned16(blob_dev) || !aligned16(ws_dev)) return TSQ_ERR_INVALID_ARG;
  const BlobLayout L = layout_for(plan, static_cast<unsigned long long>(tokens));
  if (blob_bytes < L.total || ws_bytes < plan->workspace_bytes) return TSQ_ERR_BUFFER_TOO_SMALL;
  return TSQ_OK;
}

tsq_status_t tsq_encode(const tsq_plan_t* plan, const void* x_dev, int64_t tokens, void* blob_dev, size_t blob_bytes,
                        void* ws_dev, size_t ws_bytes, void* cuda_stream) {
  const tsq_status_t args_ok = check_encode_args(plan, x_dev, tokens, blob_dev, blob_bytes, ws_dev, ws_bytes);
  if (args_ok != TSQ_OK) return args_ok;
  const BlobLayout L = layout_for(plan, static_cast<unsigned long long>(tokens));

  EncodeParams p;
  std::memset(&p, 0, sizeof p);
  p.x = static_cast<const uint16_t*>(x_dev);
  p.blob = static_cast<unsigned char*>(blob_dev);
  p.ws = static_cast<WsControl*>(ws_dev);
  p.desc = reinterpret_cast<unsigned long long*>(static_cast<unsigned char*>(ws_dev) + sizeof(WsControl));
  p.lay = L;
  p.tokens = static_cast<uint32_t>(tokens);
  p.hidden = plan->hidden;
  p.units = plan->units;
  p.chunks = plan->chunks;
  p.thr16 = plan->thr16;
  p.n_bits = plan->n_bits;
  for (int i = 0; i < 8; ++i) p.bits[i] = plan->bits[i];
  p.s_max = plan->s_max;
  p.vec_store = (plan->units % 4u == 0u) ? 1u : 0u;
  p.dtype = static_cast<uint32_t>(plan->dtype);
  p.variant = plan->variant;
  p.tau = plan->tau;
  p.delta = plan->delta;

  cudaError_t e;
  if (plan->pipe_ctas_per_sm > 0 && tokens > 2 * static_cast<int64_t>(plan->sms)) {
    // many rows: persistent CTAs that overlap the stages of consecutive rows
    p.compute_threads = plan->pipe_compute;
    p.park_stride = plan->pipe_park;
    p.planes_stride = plan->pipe_planes;
    p.csr_cap = plan->pipe_csr_cap;
    p.ring = plan->pipe_ring;
    const long long resident = static_cast<long long>(plan->sms) * plan->pipe_ctas_per_sm;
    const int grid = static_cast<int>(tokens < resident ? tokens : resident);
    e = launch_encode_pipe(p, plan->pipe_full, grid, plan->pipe_threads, plan->pipe_smem, static_cast<cudaStream_t>(cuda_stream));
  } else {
    // few rows (or rows too long for the pipeline): one CTA per row; a call without rows still launches
    // one CTA, which writes the header
    const int grid = tokens > 0 ? static_cast<int>(tokens) : 1;
    // up to one CTA per SM is resident whatever the CTA's size: such a call needs no tickets
    p.direct_tiles = tokens <= static_cast<int64_t>(plan->sms) ? 1u : 0u;
    e = launch_encode_rows(p, grid, plan->enc_threads, plan->enc_upt, static_cast<cudaStream_t>(cuda_stream));
  }
  g_launches.fetch_add(1);
  return e == cudaSuccess ? TSQ_OK : TSQ_ERR_CUDA;
}

tsq_status_t tsq_decode(const tsq_plan_t* plan, const void* blob_dev, size_t blob_bytes, int64_t tokens, void* y_dev,
                        void* ws_dev, size_t ws_bytes, void* cuda_stream) {
  if (!plan || !blob_dev || !ws_dev || tokens < 0 || static_cast<unsigned long long>(tokens) > plan->max_tokens)
    return TSQ_ERR_INVALID_ARG;
  if (tokens > 0 && !y_dev) return TSQ_ERR_INVALID_ARG;
  if (!aligned16(y_dev) || !aligned16(blob_dev) || !aligned16(ws_dev)) return TSQ_ERR_INVALID_ARG;
  const BlobLayout L = layout_for(plan, static_cast<unsigned long long>(tokens));
  if (blob_bytes < L.total || ws_bytes < plan->workspace_bytes) return TSQ_ERR_BUFFER_TOO_SMALL;
  if (tokens == 0) return TSQ_OK;

  DecodeParams p;
  std::memset(&p, 0, sizeof p);
  p.blob = static_cast<const unsigned char*>(blob_dev);
  p.y = static_cast<uint16_t*>(y_dev);
  p.ws = static_cast<WsControl*>(ws_dev);
  p.lay = L;
  p.tokens = static_cast<uint32_t>(tokens);
  p.hidden = plan->hidden;
  p.units = plan->units;
  p.chunks = plan->chunks;
  p.bmax = static_cast<uint32_t>(plan->bmax);
  p.dtype = static_cast<uint32_t>(plan->dtype);
  p.variant = plan->variant;
  p.blob_bytes = blob_bytes;
  const bool many_rows = tokens >= 3 * static_cast<int64_t>(plan->sms) * plan->dec_blocks_half;
  const cudaError_t e = launch_decode(p, static_cast<int>(tokens), many_rows ? plan->threads_half : plan->threads,
                                      plan->dec_smem, static_cast<cudaStream_t>(cuda_stream));
  g_launches.fetch_add(1);
  return e == cudaSuccess ? TSQ_OK : TSQ_ERR_CUDA;
}

tsq_status_t tsq_encode_noalloc(const tsq_plan_t* plan, const void* x_dev, int64_t tokens, void* blob_dev,
                                size_t blob_bytes, void* cuda_stream) {
  if (!plan) return TSQ_ERR_INVALID_ARG;
  if (plan->max_tokens > kStaticMaxTokens || plan->workspace_bytes > kStaticWsBytes) return TSQ_ERR_UNSUPPORTED;
  // the stream (and the kernels launched on it) belong to the current device: it has to be the plan's
  int current = -1;
  if (cudaGetDevice(&current) != cudaSuccess) {
    cudaGetLastError();
    return TSQ_ERR_CUDA;
  }
  if (current != plan->device) return TSQ_ERR_INVALID_ARG;
  void* ws = nullptr;
  if (static_workspace(plan->device, &ws) != cudaSuccess) {
    cudaGetLastError();
    return TSQ_ERR_CUDA;
  }
  // every argument error is reported before the shared array is touched
  const tsq_status_t args_ok = check_encode_args(plan, x_dev, tokens, blob_dev, blob_bytes, ws, kStaticWsBytes);
  if (args_ok != TSQ_OK) return args_ok;
  // The array keeps whatever the last call left (including an unfinished call's tickets): start clean.
  // This also zeroes the generation counter and the recorded capacity: every call through this entry
  // point runs as generation 1, so the wrap-around path that reads the capacity is never taken here.
  if (cudaMemsetAsync(ws, 0, plan->workspace_bytes, static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) {
    cudaGetLastError();
    return TSQ_ERR_CUDA;
  }
  return tsq_encode(plan, x_dev, tokens, blob_dev, blob_bytes, ws, kStaticWsBytes, cuda_stream);
}

static unsigned long long payload_of(unsigned long long tokens, unsigned long long words, unsigned long long outliers) {
  return 64ull + 9ull * tokens + 8ull * (tokens + 1ull) + 4ull * words + 4ull * outliers;
}

tsq_status_t tsq_blob_info(const void* blob_dev, tsq_info_t* out, void* cuda_stream) {
  if (!blob_dev || !out) return TSQ_ERR_INVALID_ARG;
  BlobHeader h;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemcpyAsync(&h, blob_dev, sizeof h, cudaMemcpyDeviceToHost, st) != cudaSuccess) return TSQ_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return TSQ_ERR_CUDA;
  if (h.magic != kMagic || h.version != kVersion) return TSQ_ERR_CORRUPT_BLOB;
  out->status = h.status;
  out->tokens = h.tokens;
  out->hidden = h.hidden;
  out->dtype = h.dtype;
  out->total_words = h.total_words;
  out->total_outliers = h.total_outliers;
  const unsigned long long stored = h.total_outliers < h.outlier_capacity ? h.total_outliers : h.outlier_capacity;
  out->payload_bytes = payload_of(h.tokens, h.total_words, stored);
  return TSQ_OK;
}

tsq_status_t tsq_workspace_status(const void* ws_dev, uint32_t* encode_status, uint32_t* decode_status,
                                  void* cuda_stream) {
  if (!ws_dev) return TSQ_ERR_INVALID_ARG;
  WsControl c;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemcpyAsync(&c, ws_dev, sizeof c, cudaMemcpyDeviceToHost, st) != cudaSuccess) return TSQ_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return TSQ_ERR_CUDA;
  if (encode_status) *encode_status = c.enc_status;
  if (decode_status) *decode_status = c.dec_status;
  return TSQ_OK;
}

tsq_status_t tsq_encode_host(const tsq_plan_t* plan, const void* x_host, int64_t tokens, void* blob_host,
                             size_t blob_bytes, uint64_t* payload_bytes, void* x_dev, void* blob_dev, void* ws_dev,
                             size_t ws_bytes, void* cuda_stream) {
  if (!plan || !blob_host || !blob_dev || !ws_dev || tokens < 0) return TSQ_ERR_INVALID_ARG;
  if (tokens > 0 && (!x_host || !x_dev)) return TSQ_ERR_INVALID_ARG;
  if (static_cast<unsigned long long>(tokens) > plan->max_tokens) return TSQ_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const BlobLayout L = layout_for(plan, static_cast<unsigned long long>(tokens));
  if (blob_bytes < L.total) return TSQ_ERR_BUFFER_TOO_SMALL;
  const size_t x_bytes = static_cast<size_t>(tokens) * plan->hidden * 2u;
  if (x_bytes && cudaMemcpyAsync(x_dev, x_host, x_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return TSQ_ERR_CUDA;
  const tsq_status_t s = tsq_encode(plan, x_dev, tokens, blob_dev, blob_bytes, ws_dev, ws_bytes, cuda_stream);
  if (s != TSQ_OK) return s;
  // header and per-token fields first: they say how much of the planes and of the CSR list is in use
  unsigned char* bh = static_cast<unsigned char*>(blob_host);
  const unsigned char* bd = static_cast<const unsigned char*>(blob_dev);
  if (cudaMemcpyAsync(bh, bd, static_cast<size_t>(L.off_words), cudaMemcpyDeviceToHost, st) != cudaSuccess) return TSQ_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return TSQ_ERR_CUDA;
  BlobHeader h;
  std::memcpy(&h, bh, sizeof h);
  if (h.magic != kMagic) return TSQ_ERR_CORRUPT_BLOB;
  const unsigned long long stored = h.total_outliers < L.outlier_capacity ? h.total_outliers : L.outlier_capacity;
  if (h.total_words > L.words_capacity) return TSQ_ERR_CORRUPT_BLOB;
  if (h.total_words && cudaMemcpyAsync(bh + L.off_words, bd + L.off_words, static_cast<size_t>(4 * h.total_words),
                                       cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return TSQ_ERR_CUDA;
  if (stored && cudaMemcpyAsync(bh + L.off_outl, bd + L.off_outl, static_cast<size_t>(4 * stored), cudaMemcpyDeviceToHost,
                                st) != cudaSuccess)
    return TSQ_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return TSQ_ERR_CUDA;
  if (payload_bytes) *payload_bytes = payload_of(h.tokens, h.total_words, stored);
  return static_cast<tsq_status_t>(h.status);
}

tsq_status_t tsq_decode_host(const tsq_plan_t* plan, const void* blob_host, size_t blob_bytes, int64_t tokens,
                             void* y_host, void* blob_dev, void* y_dev, void* ws_dev, size_t ws_bytes,
                             void* cuda_stream) {
  if (!plan || !blob_host || !blob_dev || !ws_dev || tokens < 0) return TSQ_ERR_INVALID_ARG;
  if (tokens > 0 && (!y_host || !y_dev)) return TSQ_ERR_INVALID_ARG;
  if (static_cast<unsigned long long>(tokens) > plan->max_tokens) return TSQ_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const BlobLayout L = layout_for(plan, static_cast<unsigned long long>(tokens));
  if (blob_bytes < L.total) return TSQ_ERR_BUFFER_TOO_SMALL;
  BlobHeader h;
  std::memcpy(&h, blob_host, sizeof h);
  if (h.magic != kMagic || h.version != kVersion || h.tokens != static_cast<uint32_t>(tokens) ||
      h.total_words > L.words_capacity)
    return TSQ_ERR_CORRUPT_BLOB;
  const unsigned long long stored = h.total_outliers < L.outlier_capacity ? h.total_outliers : L.outlier_capacity;
  const unsigned char* bh = static_cast<const unsigned char*>(blob_host);
  unsigned char* bd = static_cast<unsigned char*>(blob_dev);
  if (cudaMemcpyAsync(bd, bh, static_cast<size_t>(L.off_words), cudaMemcpyHostToDevice, st) != cudaSuccess) return TSQ_ERR_CUDA;
  if (h.total_words && cudaMemcpyAsync(bd + L.off_words, bh + L.off_words, static_cast<size_t>(4 * h.total_words),
                                       cudaMemcpyHostToDevice, st) != cudaSuccess)
    return TSQ_ERR_CUDA;
  if (stored && cudaMemcpyAsync(bd + L.off_outl, bh + L.off_outl, static_cast<size_t>(4 * stored), cudaMemcpyHostToDevice,
                                st) != cudaSuccess)
    return TSQ_ERR_CUDA;
  const tsq_status_t s = tsq_decode(plan, blob_dev, blob_bytes, tokens, y_dev, ws_dev, ws_bytes, cuda_stream);
  if (s != TSQ_OK) return s;
  const size_t y_bytes = static_cast<size_t>(tokens) * plan->hidden * 2u;
  if (y_bytes && cudaMemcpyAsync(y_host, y_dev, y_bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) return TSQ_ERR_CUDA;
  uint32_t dec = 0;
  const tsq_status_t ws = tsq_workspace_status(ws_dev, nullptr, &dec, cuda_stream);
  if (ws != TSQ_OK) return ws;
  return static_cast<tsq_status_t>(dec);
}

}  // extern "C"
