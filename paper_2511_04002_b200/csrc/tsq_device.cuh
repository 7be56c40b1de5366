// Device-side helpers of the tsq kernels: PTX wrappers (mbarrier, bulk async copies, relaxed
// global accesses), packed 16-bit operations for fp16 / bf16, and the 8x32 bit-matrix transpose
// that turns 32 byte-codes into 8 bit-plane words (and back).
#ifndef TSQ_DEVICE_CUH_
#define TSQ_DEVICE_CUH_

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>
#include <string.h>

namespace tsq {

constexpr uint32_t kFull = 0xffffffffu;

// ---- shared-memory barriers and bulk copies -------------------------------------------------

__device__ __forceinline__ uint32_t smem_addr(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_fence_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes)
               : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_addr(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}

// Wait for a phase of the barrier with an iteration limit; false = gave up.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, uint32_t limit) {
  for (uint32_t i = 0; i < limit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
  }
  return false;
}

// Global -> shared bulk copy (bytes % 16 == 0, both addresses 16-byte aligned), completion
// signalled on the barrier as transferred bytes.
__device__ __forceinline__ void bulk_g2s(void* smem_dst, const void* gmem_src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_addr(smem_dst)),
               "l"(gmem_src), "r"(bytes), "r"(smem_addr(bar))
               : "memory");
}

// Shared -> global bulk copy, tracked by the calling thread's bulk group.
__device__ __forceinline__ void bulk_s2g(void* gmem_dst, const void* smem_src, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gmem_dst),
               "r"(smem_addr(smem_src)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_all() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
// all bulk groups of this thread but the latest have finished reading their source
__device__ __forceinline__ void bulk_wait_read_but_one() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// Per-thread asynchronous 16-byte copies global -> shared (no registers hold the data in flight).  The
// lines are kept in L1 as well: the encoder reads the patterns of a group's further outliers from the
// input a second time (measured 1 to 2 % faster than bypassing L1).
__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"(smem_addr(smem_dst)), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }

__device__ __forceinline__ unsigned long long ld_relaxed_u64(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
// two adjacent 64-bit words in one request (16-byte aligned); nothing is assumed about the pair being read atomically
__device__ __forceinline__ void ld_relaxed_u64x2(const unsigned long long* p, unsigned long long& a, unsigned long long& b) {
  asm volatile("ld.relaxed.gpu.global.v2.u64 {%0, %1}, [%2];" : "=l"(a), "=l"(b) : "l"(p) : "memory");
}
__device__ __forceinline__ void st_relaxed_u64(unsigned long long* p, unsigned long long v) {
  asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

// a * b + c as an integer multiply-add instruction (the FMA pipe), whatever a plain expression would become
__device__ __forceinline__ uint32_t mad_u32(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t r;
  asm("mad.lo.u32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(c));
  return r;
}

// ---- packed 16-bit element operations ------------------------------------------------------------

template <bool BF16>
struct Elem;

template <>
struct Elem<false> {  // IEEE binary16
  static constexpr uint32_t kInfPattern = 0x7c00u;
  // bit casts by memcpy (a pointer cast would break the aliasing rules)
  static __device__ __forceinline__ __half2 as2(uint32_t v) {
    __half2 h;
    memcpy(&h, &v, sizeof h);
    return h;
  }
  static __device__ __forceinline__ uint32_t bits(__half2 v) {
    uint32_t u;
    memcpy(&u, &v, sizeof u);
    return u;
  }
  // 0xffff in each half where a >= b or the pair is unordered
  static __device__ __forceinline__ uint32_t geu_mask(uint32_t a, uint32_t b) { return __hgeu2_mask(as2(a), as2(b)); }
  static __device__ __forceinline__ uint32_t max2(uint32_t a, uint32_t b) { return bits(__hmax2(as2(a), as2(b))); }
  static __device__ __forceinline__ uint32_t min2(uint32_t a, uint32_t b) { return bits(__hmin2(as2(a), as2(b))); }
  static __device__ __forceinline__ float lo_f32(uint32_t v) { return __low2float(as2(v)); }
  static __device__ __forceinline__ float hi_f32(uint32_t v) { return __high2float(as2(v)); }
  static __device__ __forceinline__ float pattern_f32(uint32_t p) {
    return __half2float(__ushort_as_half(static_cast<unsigned short>(p)));
  }
  // two non-negative binary32 values -> packed 16-bit, round-to-nearest-even
  static __device__ __forceinline__ uint32_t pack_rn(float lo, float hi) { return bits(__floats2half2_rn(lo, hi)); }
  // largest pattern whose value is <= f (f >= 0)
  static __device__ __forceinline__ uint32_t pattern_rd(float f) { return __half_as_ushort(__float2half_rz(f)); }
};

template <>
struct Elem<true> {  // bfloat16
  static constexpr uint32_t kInfPattern = 0x7f80u;
  static __device__ __forceinline__ __nv_bfloat162 as2(uint32_t v) {
    __nv_bfloat162 h;
    memcpy(&h, &v, sizeof h);
    return h;
  }
  static __device__ __forceinline__ uint32_t bits(__nv_bfloat162 v) {
    uint32_t u;
    memcpy(&u, &v, sizeof u);
    return u;
  }
  static __device__ __forceinline__ uint32_t geu_mask(uint32_t a, uint32_t b) { return __hgeu2_mask(as2(a), as2(b)); }
  static __device__ __forceinline__ uint32_t max2(uint32_t a, uint32_t b) { return bits(__hmax2(as2(a), as2(b))); }
  static __device__ __forceinline__ uint32_t min2(uint32_t a, uint32_t b) { return bits(__hmin2(as2(a), as2(b))); }
  static __device__ __forceinline__ float lo_f32(uint32_t v) { return __uint_as_float(mad_u32(v, 65536u, 0u)); }
  static __device__ __forceinline__ float hi_f32(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }
  static __device__ __forceinline__ float pattern_f32(uint32_t p) { return __uint_as_float(p << 16); }
  static __device__ __forceinline__ uint32_t pack_rn(float lo, float hi) { return bits(__floats2bfloat162_rn(lo, hi)); }
  static __device__ __forceinline__ uint32_t pattern_rd(float f) { return __float_as_uint(f) >> 16; }
};

// ---- 8 x 32 bit-matrix transpose -------------------------------------------------------------------
// In: r[i] holds four byte-codes, byte c = element 8c + i of a 32-element unit.
// Out: r[k] bit (8c + i) = bit k of that element's byte, i.e. r[k] is bit-plane k of the unit.
// The network swaps the 3-bit register index with the 3-bit in-byte position; it is its own inverse.
__device__ __forceinline__ void transpose8x32(uint32_t (&r)[8]) {
#pragma unroll
  for (int b = 0; b < 3; ++b) {
    const int sh = 1 << b;
    const uint32_t mask_lo = (b == 0) ? 0x55555555u : (b == 1) ? 0x33333333u : 0x0f0f0f0fu;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      if (i & sh) continue;
      const uint32_t t = ((r[i] >> sh) ^ r[i | sh]) & mask_lo;
      r[i | sh] ^= t;
      r[i] ^= t << sh;
    }
  }
}

// ---- packed binary32 arithmetic: two lanes per 64-bit register, each lane IEEE round-to-nearest-even ----
__device__ __forceinline__ uint64_t pack2f(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ uint64_t pack2u(uint32_t lo, uint32_t hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
  return r;
}
__device__ __forceinline__ void unpack2u(uint64_t v, uint32_t& lo, uint32_t& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=r"(lo), "=r"(hi) : "l"(v));
}
__device__ __forceinline__ void unpack2f(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}

// (a & mask) | (b & ~mask) in one three-input logic instruction
__device__ __forceinline__ uint32_t bit_select(uint32_t mask, uint32_t a, uint32_t b) {
  uint32_t r;
  asm("lop3.b32 %0, %1, %2, %3, 0xCA;" : "=r"(r) : "r"(mask), "r"(a), "r"(b));
  return r;
}

// The same transpose with each exchange written as two bit selections (a shift and a three-input logic
// instruction per word, the left shift as a multiplication so that it goes to the FMA pipe) instead of the
// xor-swap's five instructions.
__device__ __forceinline__ void transpose8x32_select(uint32_t (&r)[8]) {
#pragma unroll
  for (int b = 0; b < 3; ++b) {
    const int sh = 1 << b;
    const uint32_t mask_lo = (b == 0) ? 0x55555555u : (b == 1) ? 0x33333333u : 0x0f0f0f0fu;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      if (i & sh) continue;
      const uint32_t lo = r[i], hi = r[i | sh];
      r[i | sh] = bit_select(mask_lo, lo >> sh, hi);
      r[i] = bit_select(mask_lo, lo, mad_u32(hi, 1u << sh, 0u));
    }
  }
}

}  // namespace tsq

#endif  // TSQ_DEVICE_CUH_
