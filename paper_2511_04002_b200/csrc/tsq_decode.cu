// tsq decode kernel: Eq. "dequnt" — unpack the bit-planes of one token, restore
// (code + zero-point) * scale, round once to the 16-bit type, put the sign back, then write the
// outliers of T_above over their slots.  One CTA per token row; the row is assembled in shared
// memory and leaves through one bulk asynchronous store.
//
// Every field read from the blob is checked against the capacities of the call before it is used
// as an index: a malformed blob makes the kernel record TSQ_ERR_CORRUPT_BLOB and skip the row.

#include <mutex>

#include "tsq_device.cuh"
#include "tsq_internal.h"

namespace tsq {
namespace {

constexpr float kTwo23 = 8388608.0f;
constexpr uint32_t kTwo23Bits = 0x4B000000u;

__device__ __forceinline__ void record_decode_error(const DecodeParams& p, uint32_t code) {
  atomicCAS(&p.ws->dec_status, 0u, code);
}


// Unpack, dequantise and stage this thread's groups of one row.
//   DIRECT = false: float(code + zp) is formed without a conversion instruction: the pattern of
//   2^23 + n carries n in its low mantissa bits, and (2^23 + n) * s - 2^23 * s equals n * s exactly,
//   so one FMA rounds n * s once (2^23 * s is a power-of-two multiple of s, hence exact while
//   finite).  ZP0 (zero-point 0, the usual case) ORs the code into that pattern instead of adding.
//   DIRECT = true: int -> float conversion and one multiplication (scales too large for 2^23 * s).
// The integer / logic pipe is the scarce one here too: two elements travel per register, and the
// shifts that can be multiplications are written as such.
template <bool BF16, bool DIRECT, bool ZP0>
__device__ __forceinline__ void restore_units(const DecodeParams& p, const uint32_t* words, uint32_t b, float s,
                                              int32_t zp) {
  using E = Elem<BF16>;
  extern __shared__ __align__(128) unsigned char smem_dyn[];
  uint4* stage4 = reinterpret_cast<uint4*>(smem_dyn);
  const float neg_bias = DIRECT ? 0.0f : -__fmul_rn(kTwo23, s);
  const bool vec = (reinterpret_cast<uintptr_t>(words) & 15u) == 0;  // 16-byte loads of a group's words
  const uint32_t magic = kTwo23Bits + static_cast<uint32_t>(zp);
  for (uint32_t u = threadIdx.x; u < p.units; u += blockDim.x) {
    // group u owns words u * b .. u * b + b - 1: plane 0 = sign, plane 1 + k = code bit k.
    // r[k] = bit k of the bytes to come: code bits in r[0..6], signs in r[7].
    uint32_t r[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    const uint32_t* src = words + static_cast<size_t>(u) * b;
    if (vec && b == 8u) {
      const uint4 lo = __ldg(reinterpret_cast<const uint4*>(src)), hi = __ldg(reinterpret_cast<const uint4*>(src) + 1);
      r[7] = lo.x; r[0] = lo.y; r[1] = lo.z; r[2] = lo.w;
      r[3] = hi.x; r[4] = hi.y; r[5] = hi.z; r[6] = hi.w;
    } else if (vec && b == 4u) {
      const uint4 lo = __ldg(reinterpret_cast<const uint4*>(src));
      r[7] = lo.x; r[0] = lo.y; r[1] = lo.z; r[2] = lo.w;
    } else {
      r[7] = __ldg(src);
#pragma unroll
      for (int k = 0; k < 7; ++k) {
        if (static_cast<uint32_t>(k) + 1u < b) r[k] = __ldg(src + 1 + k);
      }
    }
    transpose8x32_select(r);  // r[i] byte c = (code | sign << 7) of element 8c + i
    const uint32_t rot = (u >> 1) & 3u;
#pragma unroll
    for (uint32_t j = 0; j < 4; ++j) {
      const uint32_t cc = (j + rot) & 3u;
      const uint32_t cidx = 4u * u + cc;
      if (cidx >= p.chunks) continue;
      const uint32_t sel = cc * 0x1111u + 0x4400u;  // byte cc of the first operand -> byte 0, of the second -> byte 2
      uint32_t out[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t p2 = __byte_perm(r[2 * i], r[2 * i + 1], sel);  // elements 8cc + 2i (byte 0) and 8cc + 2i + 1 (byte 2)
        if (ZP0 && !DIRECT) {
          // zero-point 0: the pattern of 2^23 + code is the code byte under the top byte of 2^23, two byte
          // permutes; both products (2^23 + code) * s - 2^23 * s in one packed FMA (each lane rounds as the
          // scalar instruction does)
          const uint32_t c2 = p2 & 0x007f007fu;
          const uint64_t v2 = pack2u(__byte_perm(c2, kTwo23Bits, 0x7440), __byte_perm(c2, kTwo23Bits, 0x7442));
          float flo2, fhi2;
          unpack2f(fma2(v2, pack2f(s, s), pack2f(neg_bias, neg_bias)), flo2, fhi2);
          out[i] = (p2 & 0x00800080u) * 256u + E::pack_rn(flo2, fhi2);  // sign bits 7 / 23 -> 15 / 31
          continue;
        }
        const uint32_t clo = p2 & 0x7fu, chi = __umulhi(p2, 65536u) & 0x7fu;
        float flo, fhi;
        if (DIRECT) {
          flo = __fmul_rn(__int2float_rn(static_cast<int>(clo) + zp), s);
          fhi = __fmul_rn(__int2float_rn(static_cast<int>(chi) + zp), s);
        } else if (ZP0) {
          flo = fmaf(__uint_as_float(clo | kTwo23Bits), s, neg_bias);
          fhi = fmaf(__uint_as_float(chi | kTwo23Bits), s, neg_bias);
        } else {
          flo = fmaf(__uint_as_float(clo + magic), s, neg_bias);
          fhi = fmaf(__uint_as_float(chi + magic), s, neg_bias);
        }
        out[i] = (p2 & 0x00800080u) * 256u + E::pack_rn(flo, fhi);  // sign bits 7 / 23 -> 15 / 31
      }
      stage4[cidx] = make_uint4(out[0], out[1], out[2], out[3]);
    }
  }
}

// The same for a blob of the signed-values variant: plane k = bit k of the code (no sign plane), the value is
// (code + zp) * s with a zero-point of either sign: conversion and one multiplication, rounded once to 16 bits.
template <bool BF16>
__device__ __noinline__ void restore_units_signed_values(const DecodeParams& p, const uint32_t* words, uint32_t b, float s,
                                                         int32_t zp) {
  using E = Elem<BF16>;
  extern __shared__ __align__(128) unsigned char smem_dyn[];
  uint4* stage4 = reinterpret_cast<uint4*>(smem_dyn);
  for (uint32_t u = threadIdx.x; u < p.units; u += blockDim.x) {
    uint32_t r[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    const uint32_t* src = words + static_cast<size_t>(u) * b;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      if (static_cast<uint32_t>(k) < b) r[k] = __ldg(src + k);
    }
    transpose8x32_select(r);  // r[i] byte c = code of element 8c + i
#pragma unroll
    for (uint32_t cc = 0; cc < 4; ++cc) {
      const uint32_t cidx = 4u * u + cc;
      if (cidx >= p.chunks) continue;
      const uint32_t sel = cc * 0x1111u + 0x4400u;
      uint32_t out[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t p2 = __byte_perm(r[2 * i], r[2 * i + 1], sel);  // elements 8cc + 2i (bytes 0, 1) and 8cc + 2i + 1 (bytes 2, 3)
        const int clo = static_cast<int>(p2 & 0xffu), chi = static_cast<int>(p2 >> 24);
        out[i] = E::pack_rn(__fmul_rn(__int2float_rn(clo + zp), s), __fmul_rn(__int2float_rn(chi + zp), s));
      }
      stage4[cidx] = make_uint4(out[0], out[1], out[2], out[3]);
    }
  }
}

template <bool BF16>
__global__ void __launch_bounds__(kMaxThreads) decode_kernel(const DecodeParams p) {
  extern __shared__ __align__(128) unsigned char smem_dyn[];  // one output row
  const uint32_t tid = threadIdx.x;
  const uint32_t t = blockIdx.x;

  // ---- header against the plan and the call ----
  const BlobHeader* h = reinterpret_cast<const BlobHeader*>(p.blob);
  if (h->magic != kMagic || h->version != kVersion) {
    if (tid == 0) record_decode_error(p, TSQ_ERR_CORRUPT_BLOB);
    return;
  }
  if (h->status != TSQ_OK) {  // the encoder flagged this blob: pass its status on
    if (tid == 0) record_decode_error(p, h->status);
    return;
  }
  const bool header_ok = h->dtype == p.dtype && h->hidden == p.hidden && h->tokens == p.tokens && h->n_bits >= 1u &&
                         h->n_bits <= static_cast<uint32_t>(kMaxCand) && h->bits[(h->n_bits - 1u) & 7u] == p.bmax &&
                         h->bits[7] == p.variant &&
                         h->outlier_capacity == static_cast<uint32_t>(p.lay.outlier_capacity) &&
                         h->total_words <= p.lay.words_capacity && h->total_outliers <= p.lay.outlier_capacity;
  if (!header_ok) {
    if (tid == 0) record_decode_error(p, TSQ_ERR_CORRUPT_BLOB);
    return;
  }

  // ---- this token's fields ----
  const uint32_t b = reinterpret_cast<const uint8_t*>(p.blob + p.lay.off_bits)[t];
  const float s = reinterpret_cast<const float*>(p.blob + p.lay.off_scale)[t];
  const int32_t zp = reinterpret_cast<const int32_t*>(p.blob + p.lay.off_zp)[t];
  const uint32_t wo = reinterpret_cast<const uint32_t*>(p.blob + p.lay.off_word_off)[t];
  const uint32_t wo_next = reinterpret_cast<const uint32_t*>(p.blob + p.lay.off_word_off)[t + 1];
  const uint32_t p0 = reinterpret_cast<const uint32_t*>(p.blob + p.lay.off_out_ptr)[t];
  const uint32_t p1 = reinterpret_cast<const uint32_t*>(p.blob + p.lay.off_out_ptr)[t + 1];
  const unsigned long long span = static_cast<unsigned long long>(b) * p.lay.wpp;
  const bool row_ok = b >= 2u && b <= p.bmax && wo + span <= h->total_words && wo_next == wo + span && p0 <= p1 &&
                      p1 <= h->total_outliers && (p1 - p0) <= p.hidden && zp < (1 << 22) &&
                      zp >= (p.variant != 0u ? 1 - (1 << 22) : 0);
  if (!row_ok) {
    if (tid == 0) record_decode_error(p, TSQ_ERR_CORRUPT_BLOB);
    return;
  }

  const uint32_t* words = reinterpret_cast<const uint32_t*>(p.blob + p.lay.off_words) + wo;
  // 2^23 * s must stay finite for the conversion-free path; huge scales take the plain one.
  if (p.variant != 0u) {
    restore_units_signed_values<BF16>(p, words, b, s, zp);
  } else if (s > 0x1p100f) {
    restore_units<BF16, true, false>(p, words, b, s, zp);
  } else if (zp == 0) {
    restore_units<BF16, false, true>(p, words, b, s, zp);
  } else {
    restore_units<BF16, false, false>(p, words, b, s, zp);
  }
  __syncthreads();

  // ---- "+ T_above": each outlier slot decoded to +0, so adding equals overwriting ----
  if (p1 != p0) {
    const uint32_t* outl = reinterpret_cast<const uint32_t*>(p.blob + p.lay.off_outl);
    uint16_t* stage16 = reinterpret_cast<uint16_t*>(smem_dyn);
    bool bad = false;
    for (uint32_t q = p0 + tid; q < p1; q += blockDim.x) {
      const uint32_t e = __ldg(outl + q);
      const uint32_t col = e >> 16;
      if (col < p.hidden) {
        stage16[col] = static_cast<uint16_t>(e & 0xffffu);
      } else {
        bad = true;
      }
    }
    if (bad) record_decode_error(p, TSQ_ERR_CORRUPT_BLOB);
    __syncthreads();
  }

  // ---- the row leaves in one bulk store ----
  if (tid == 0) {
    fence_proxy_async_smem();
    bulk_s2g(p.y + static_cast<size_t>(t) * p.hidden, smem_dyn, p.hidden * 2u);
    bulk_commit();
    bulk_wait_read_all();
  }
}

}  // namespace

size_t decode_smem_bytes(uint32_t row_bytes) { return (static_cast<size_t>(row_bytes) + 127u) & ~static_cast<size_t>(127u); }

cudaError_t decode_kernel_attrs(bool bf16, int threads, size_t smem, int* blocks_per_sm) {
  const void* fn = bf16 ? reinterpret_cast<const void*>(&decode_kernel<true>)
                        : reinterpret_cast<const void*>(&decode_kernel<false>);
  // the attribute belongs to the kernel on the current device, not to a plan: it only ever grows, so
  // that every plan can launch
  static std::mutex mu;
  static size_t granted[kMaxDevices][2] = {};
  {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(mu);
    if (smem > granted[dev][bf16 ? 1 : 0]) {
      e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
      if (e != cudaSuccess) return e;
      granted[dev][bf16 ? 1 : 0] = smem;
    }
  }
  return cudaOccupancyMaxActiveBlocksPerMultiprocessor(blocks_per_sm, fn, threads, smem);
}

cudaError_t launch_decode(const DecodeParams& p, int grid, int threads, size_t smem, cudaStream_t stream) {
  if (p.dtype == TSQ_BF16) {
    decode_kernel<true><<<grid, threads, smem, stream>>>(p);
  } else {
    decode_kernel<false><<<grid, threads, smem, stream>>>(p);
  }
  return cudaGetLastError();
}

}  // namespace tsq
