// tsq encode kernels: threshold splitting (Eq. "ts") + token-wise TAB-Q (Algorithm 1 on AIQ,
// Eq. "Proposed") + bit-plane packing + CSR emission, fused into one kernel.
//
// One CTA encodes one token row at a time, one thread per group of 32 elements (64 bytes), and every
// thread only ever touches its own group: the input is read from HBM exactly once.  The passes:
//   A  threshold split: outlier bitmap, outlier slots set to +0 (what T_below holds there), and
//      the row's min / max of the inlier magnitudes (CTA reduction);
//   B  Algorithm 1: AIQ codes at the top level and at each lower candidate, distortion sums
//      (CTA reduction, one candidate at a time, stopping at the first failure);
//   C  codes at the chosen level -> bytes (code | sign << 7) -> 8 x 32 bit transpose -> the
//      group's b* plane words, one contiguous run per thread.
// Between the passes sits scalar work per row (the AIQ parameters of every candidate: a few
// divisions) and the placement of the row's output, which has to wait for every earlier row.
//
// Two kernels share the passes:
//   encode_rows_kernel  one CTA per row, the group in registers from load to store, everything in
//                       order; used for few rows (lowest latency per call) and for rows longer
//                       than the pipelined kernel takes.
//   encode_pipe_kernel  persistent CTAs that keep several rows in different stages at once, so that
//                       the vector passes never wait for the scalar work or for the placement.
//                       Each compute thread copies its group of the next row into shared memory
//                       asynchronously (no registers held), runs pass A on row n in place there,
//                       then passes B and C of row n - 1 from its copy; a "levels" warp turns row
//                       n's min / max into AIQ parameters meanwhile; a "placement" warp resolves the
//                       offsets of rows packed earlier, ships their planes with one bulk
//                       asynchronous store each and writes their CSR entries.  When the first
//                       lower candidate fails (the usual case) pass C reuses the top-level bytes
//                       that pass B already formed.
//
// The binding resource is the integer / logic pipe, which issues at half the rate of the FMA pipe:
// the passes work on two 16-bit elements per 32-bit register wherever they can (four codes as bytes
// in the distortion sum and on the way to the bit transpose), and some shifts and merges are written
// as integer multiply-adds so that they go to the FMA pipe instead.
//
// Variable-length placement: where a token's planes and CSR entries start is an exclusive prefix
// sum over all earlier tokens.  It is resolved with a decoupled look-back over per-token
// descriptors in the workspace.  Rows are numbered by an atomic ticket taken by a running CTA,
// so a row only ever waits for rows whose CTAs are already running, and a row publishes its own
// sizes before it waits for anything.  A look-back step reads 256 descriptor pairs at once (eight
// independent loads per lane) in the one-CTA-per-row kernel and 32 in the pipelined kernel.  Every wait
// is bounded and fails into a status word.
//
// Arithmetic contract: the codes equal  clamp(rint(m / s) - zp, 0, Qmax)  with the IEEE binary32
// quotient m / s.  "Plain" rows (nearly every row of real data: zero-point 0, which any row with an
// outlier or a tiny element has; no code above Qmax; scale in [2^-60, 2^60], so that no intermediate
// leaves the normal range) form the quotient without the division instruction: r = fl(1 / s) once
// per row and level, then per element q0 = fl(m * r), the residual m - q0 * s (one FMA) and
// q = fl(q0 + residual * r), two elements at a time with the packed binary32 instructions (each
// lane rounds to nearest even, as the scalar instructions do).  rint is one addition of 2^23, and
// the code is the low byte of the sum's pattern: no subtraction, no clamp.  What has to hold is
// that rint(q) equals rint(fl(m / s)) for every 16-bit magnitude m of the row; a host-side test
// checks the three-operation sequence in exact arithmetic against the true quotient for every
// 16-bit pattern over many ranges and levels, and the GPU parity tests compare every code.  (A
// single fl(m * r) is not enough: 16-bit inputs put m / s on or next to a rounding boundary
// k + 1/2 in almost every row, and there the two can round differently.)  Every other row goes
// through the division instruction in compact loops.

#include <mutex>

#include "tsq_device.cuh"
#include "tsq_internal.h"

namespace tsq {
namespace {

constexpr float kRoundMagic = 8388608.0f;  // 2^23: adding it to 0 <= y < 2^23 rounds y to an integer, ties to even
constexpr uint32_t kLookbackPollLimit = 1u << 20;  // polls of one descriptor (200 ns to 1 us apart): about a second
constexpr uint32_t kHandshakeFactor = 4u;          // handshakes inside a CTA poll faster: four times as many polls

// AIQ parameters of one candidate level for one row (Eq. "Proposed").
struct __align__(16) Level {
  float s;    // scale
  float r;    // fl(1 / s)
  int zp;     // zero-point rint(m_min / s)
  int qmax;   // 2^(b-1) - 1
};

// *plain: the fast steps apply to the level: FMA quotient safe, zero-point 0, no code needs the clamp (see the file header).
__device__ __forceinline__ Level make_level(float mmin, float mmax, int b, bool* plain) {
  Level c;
  c.qmax = (1 << (b - 1)) - 1;
  const float range = __fsub_rn(mmax, mmin);
  c.s = range > 0.0f ? __fdiv_rn(range, static_cast<float>(c.qmax)) : (mmax > 0.0f ? mmax : 1.0f);
  c.zp = mmin > 0.0f ? __float2int_rn(__fdiv_rn(mmin, c.s)) : 0;  // 0 / s = 0: the usual row needs no division here
  c.r = __frcp_rn(c.s);
  // Plain: no intermediate of the FMA quotient can leave the normal range, the zero-point is 0 (so no code is
  // negative) and the largest magnitude's code needs no clamp (codes grow with the magnitude).  With a minimum
  // of 0 the scale is fl(max / Qmax) and max / scale rounds to Qmax: no division needed to know.
  *plain = (c.s >= 0x1p-60f) && (c.s <= 0x1p60f) && c.zp == 0 &&
           (mmin == 0.0f || __float2int_rn(__fdiv_rn(mmax, c.s)) <= c.qmax);
  return c;
}

// The signed-values variant (Eq. "Proposed" on the signed inliers): Q_max = 2^b - 1, the zero-point may be
// negative, a constant row takes its own magnitude as the scale.  *plain: the fast steps apply: the FMA quotient is
// safe and no code needs a clamp (codes grow with the value, the smallest is 0 by construction, so the largest
// value's code decides); the zero-point is then subtracted byte-wise, modulo 256.
__device__ __forceinline__ Level make_level_signed(float vmin, float vmax, int b, bool* plain) {
  Level c;
  c.qmax = (1 << b) - 1;
  // two finite values of opposite sign can lie further apart than binary32 holds: the largest finite value then
  const float range = fminf(__fsub_rn(vmax, vmin), 3.40282346638528859811704183484516925e+38f);
  const float a = fabsf(vmax);
  c.s = range > 0.0f ? __fdiv_rn(range, static_cast<float>(c.qmax)) : (a > 0.0f ? a : 1.0f);
  c.zp = __float2int_rn(__fdiv_rn(vmin, c.s));
  c.r = __frcp_rn(c.s);
  *plain = (c.s >= 0x1p-60f) && (c.s <= 0x1p60f) && (__float2int_rn(__fdiv_rn(vmax, c.s)) - c.zp <= c.qmax);
  return c;
}

// 16-bit patterns of signed values <-> 16-bit keys that order like the values (-0 just below +0).
__device__ __forceinline__ uint32_t order_keys2(uint32_t v2) {
  return v2 ^ 0x80008000u ^ (((v2 >> 15) & 0x10001u) * 0x7fffu);
}
__device__ __forceinline__ uint32_t pattern_of_key(uint32_t key) { return (key & 0x8000u) ? key ^ 0x8000u : key ^ 0xffffu; }

// Codes of the two elements of a 16-bit pair, as two 16-bit integers, by the division instruction: for rows
// that are not plain.  SV = false: codes of the magnitudes (sign bits ignored); SV = true: of the signed values.
template <bool BF16, bool SV = false>
__device__ __forceinline__ uint32_t codes2_divide(uint32_t x, const Level& c) {
  using E = Elem<BF16>;
  const float lo = SV ? E::lo_f32(x) : fabsf(E::lo_f32(x)), hi = SV ? E::hi_f32(x) : fabsf(E::hi_f32(x));
  const int klo = __vimin_s32_relu(__float2int_rn(__fdiv_rn(lo, c.s)) - c.zp, c.qmax);
  const int khi = __vimin_s32_relu(__float2int_rn(__fdiv_rn(hi, c.s)) - c.zp, c.qmax);
  return static_cast<uint32_t>(klo) | (static_cast<uint32_t>(khi) << 16);
}

// ---- plain rows: two elements at a time with the packed binary32 instructions (each lane IEEE round-to-nearest-even) ----
struct Level2 {
  uint64_t r2, ns2;  // {r, r} and {-s, -s}
  uint32_t zp4;      // signed-values variant: the zero-point modulo 256 in every byte
};
__device__ __forceinline__ Level2 make_level2(const Level& c) {
  Level2 l;
  l.r2 = pack2f(c.r, c.r);
  l.ns2 = pack2f(-c.s, -c.s);
  l.zp4 = (static_cast<uint32_t>(c.zp) & 0xffu) * 0x01010101u;
  return l;
}
// Magnitudes of the two elements of a 16-bit pair as packed binary32.
template <bool BF16>
__device__ __forceinline__ uint64_t magnitudes2(uint32_t x) {
  const uint32_t a = x & 0x7fff7fffu;
  if (BF16) return pack2u(mad_u32(a, 65536u, 0u), a & 0xffff0000u);
  const float2 f = __half22float2(Elem<false>::as2(a));
  return pack2f(f.x, f.y);
}
// rint(fl(m / s)) + 2^23 in both lanes: q0 = fl(m r), the residual m - q0 s (one FMA, exact), q = fl(q0 + residual r),
// then the addition that rounds to an integer.  The code is the low byte of the result's pattern.
__device__ __forceinline__ uint64_t quotient2(uint64_t m2, const Level2& l, uint64_t magic2) {
  const uint64_t q0 = mul2(m2, l.r2);
  const uint64_t e = fma2(q0, l.ns2, m2);
  const uint64_t q = fma2(e, l.r2, q0);
  return add2(q, magic2);
}
// Low bytes of four patterns 2^23 + k (k < 256) as one word: bytes a.lo, b.lo, a.hi, b.hi.
__device__ __forceinline__ uint32_t bytes4(uint64_t ta, uint64_t tb) {
  uint32_t alo, ahi, blo, bhi;
  unpack2u(ta, alo, ahi);
  unpack2u(tb, blo, bhi);
  return __byte_perm(mad_u32(blo, 256u, alo), mad_u32(bhi, 256u, ahi), 0x5410);
}

// 2^23 rounds a non-negative quotient to an integer; 2^23 + 2^22 does the same for |quotient| < 2^22 of either sign
// and leaves the integer, modulo 2^22, in the low bits of the pattern (two's complement).
constexpr float kRoundMagicSigned = 12582912.0f;
// The signed values of the two elements of a 16-bit pair as packed binary32 (signed-values variant).
template <bool BF16>
__device__ __forceinline__ uint64_t values2(uint32_t x) {
  if (BF16) return pack2u(mad_u32(x, 65536u, 0u), x & 0xffff0000u);
  const float2 f = __half22float2(Elem<false>::as2(x));
  return pack2f(f.x, f.y);
}
// Low bytes of four patterns as one word (bytes a.lo, b.lo, a.hi, b.hi) when the patterns' other bytes are not
// zero (a negative rounded quotient): byte permutes only.
__device__ __forceinline__ uint32_t bytes4_any(uint64_t ta, uint64_t tb) {
  uint32_t alo, ahi, blo, bhi;
  unpack2u(ta, alo, ahi);
  unpack2u(tb, blo, bhi);
  return __byte_perm(__byte_perm(alo, blo, 0x0040), __byte_perm(ahi, bhi, 0x0040), 0x5410);
}
// The codes of four elements (pairs xa, xb) at level l as bytes a.lo, b.lo, a.hi, b.hi.  SV: of the signed values,
// zero-point subtracted modulo 256 (exact for a plain level: every code lies in [0, 255]).
template <bool BF16, bool SV>
__device__ __forceinline__ uint32_t codes4(uint32_t xa, uint32_t xb, const Level2& l) {
  if (SV) {
    const uint64_t magic2 = pack2f(kRoundMagicSigned, kRoundMagicSigned);
    return __vsub4(bytes4_any(quotient2(values2<BF16>(xa), l, magic2), quotient2(values2<BF16>(xb), l, magic2)), l.zp4);
  }
  const uint64_t magic2 = pack2f(kRoundMagic, kRoundMagic);
  return bytes4(quotient2(magnitudes2<BF16>(xa), l, magic2), quotient2(magnitudes2<BF16>(xb), l, magic2));
}

__device__ __forceinline__ uint32_t max_s16x2(uint32_t a, uint32_t b) {
  uint32_t r;
  asm("max.s16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
  return r;
}
__device__ __forceinline__ uint32_t min_s16x2(uint32_t a, uint32_t b) {
  uint32_t r;
  asm("min.s16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
  return r;
}

// Pass A on one group held in x[16] (pair i of chunk j in x[4j + i]; chunks j >= nvalid lie past the
// end of the row and hold zeros): outlier slots become +0, bit e of the result flags element e of
// the group, mn2 / mx2 collect the inlier magnitudes.
template <bool BF16>
__device__ __forceinline__ uint32_t split_group(uint32_t (&x)[16], uint32_t nvalid, uint32_t thr2, uint32_t& mn2,
                                                uint32_t& mx2) {
  using E = Elem<BF16>;
  uint32_t bitmap = 0u;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    if (static_cast<uint32_t>(j) >= nvalid) continue;
    uint32_t acc = 0u;  // bit 2i / bit 17 + 2i flag the low / high element of pair i
    uint32_t m2[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const uint32_t a = x[4 * j + i] & 0x7fff7fffu;
      const uint32_t mk = E::geu_mask(a, thr2);  // 0xffff in each half with |x| >= tau, NaN included
      m2[i] = a & ~mk;
      x[4 * j + i] &= ~mk;
      acc |= mk & ((1u << (2 * i)) | (1u << (17 + 2 * i)));
    }
    // patterns of non-negative values order like the values: integer min / max
    mx2 = __vimax3_u16x2(mx2, m2[0], m2[1]);
    mx2 = __vimax3_u16x2(mx2, m2[2], m2[3]);
    mn2 = __vimin3_u16x2(mn2, m2[0], m2[1]);
    mn2 = __vimin3_u16x2(mn2, m2[2], m2[3]);
    bitmap |= ((acc | (acc >> 16)) & 0xffu) << (8 * j);
  }
  return bitmap;
}

// Pass B on one group of a plain row: sum |(q0 >> sh) - q| over its 32 elements (Algorithm 1's distortion
// numerator).  Four codes travel as the bytes of one word: the shift and mask take four at a time, and the
// byte-wise sum-of-absolute-differences instruction adds the four differences.
// SV (signed-values variant): 8-bit codes of the signed values; the chunks at and past `nvalid` lie beyond the end
// of the row and do not count (their zeros would get the code of the value 0, which is not 0 there).
template <bool BF16, bool SV = false>
__device__ __forceinline__ uint32_t distortion_group(const uint32_t (&x)[16], const Level2& top, const Level2& low, int sh,
                                                     uint32_t nvalid = 4u) {
  const uint32_t shmask = ((SV ? 0xffu : 0x7fu) >> sh) * 0x01010101u;
  const uint64_t magic2 = pack2f(kRoundMagic, kRoundMagic);
  uint32_t S = 0;
#pragma unroll
  for (int i = 0; i < 16; i += 2) {
    if (SV) {
      if (static_cast<uint32_t>(i / 4) >= nvalid) continue;
      S = __vsadu4((codes4<BF16, true>(x[i], x[i + 1], top) >> sh) & shmask, codes4<BF16, true>(x[i], x[i + 1], low)) + S;
      continue;
    }
    const uint64_t ma = magnitudes2<BF16>(x[i]), mb = magnitudes2<BF16>(x[i + 1]);
    const uint32_t ct4 = bytes4(quotient2(ma, top, magic2), quotient2(mb, top, magic2));
    const uint32_t q4 = bytes4(quotient2(ma, low, magic2), quotient2(mb, low, magic2));
    S = __vsadu4((ct4 >> sh) & shmask, q4) + S;
  }
  return S;
}

// Pass B for the first lower candidate, keeping what pass C needs if that candidate fails: on return tb[4h + i]
// holds the top-level bytes (code | sign << 7) of elements 16h + 2i, 16h + 8 + 2i, 16h + 2i + 1, 16h + 8 + 2i + 1 (pair i
// of chunks 2h and 2h + 1, low elements first) and ql the candidate's own codes in the same grouping, no signs.
// (Any grouping of four serves the sum; this one costs the byte assembly least, and two byte permutes per i
// turn it into the input of the bit transpose.)
// SV: bytes are the 8-bit codes of the signed values, no signs; bytes of chunks at and past `nvalid` are 0.
template <bool BF16, bool SV = false>
__device__ __forceinline__ uint32_t distortion_first(const uint32_t (&x)[16], const Level2& top, const Level2& low, int sh,
                                                     uint32_t (&tb)[8], uint32_t (&ql)[8], uint32_t nvalid = 4u) {
  const uint32_t shmask = ((SV ? 0xffu : 0x7fu) >> sh) * 0x01010101u;
  const uint64_t magic2 = pack2f(kRoundMagic, kRoundMagic);
  uint32_t S = 0;
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    // bytes 0 and 2 of a word belong to chunk 2h, bytes 1 and 3 to chunk 2h + 1
    const uint32_t inside = (2u * h < nvalid ? 0x00ff00ffu : 0u) | (2u * h + 1u < nvalid ? 0xff00ff00u : 0u);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const uint32_t xa = x[8 * h + i], xb = x[8 * h + 4 + i];  // pairs i of chunks 2h and 2h + 1
      if (SV) {
        const uint32_t ct4 = codes4<BF16, true>(xa, xb, top) & inside, q4 = codes4<BF16, true>(xa, xb, low) & inside;
        S = __vsadu4((ct4 >> sh) & shmask, q4) + S;
        tb[4 * h + i] = ct4;
        ql[4 * h + i] = q4;
        continue;
      }
      const uint64_t ma = magnitudes2<BF16>(xa), mb = magnitudes2<BF16>(xb);
      const uint32_t ct4 = bytes4(quotient2(ma, top, magic2), quotient2(mb, top, magic2));
      const uint32_t q4 = bytes4(quotient2(ma, low, magic2), quotient2(mb, low, magic2));
      S = __vsadu4((ct4 >> sh) & shmask, q4) + S;
      tb[4 * h + i] = ct4 | (__byte_perm(xa, xb, 0x7351) & 0x80808080u);  // the sign bits sit in bytes 1 and 3 of a pair
      ql[4 * h + i] = q4;
    }
  }
  return S;
}

// Pass B for a further candidate: the top-level codes come from the bytes the first turn left.
template <bool BF16, bool SV = false>
__device__ __forceinline__ uint32_t distortion_next(const uint32_t (&x)[16], const uint32_t (&tb)[8], const Level2& low, int sh,
                                                    uint32_t (&ql)[8], uint32_t nvalid = 4u) {
  // a byte of tb is code | sign << 7 (SV: an 8-bit code): shifted right by sh >= 1, the sign bit and the bits that
  // come in from the next byte all land above the mask
  const uint32_t shmask = ((SV ? 0xffu : 0x7fu) >> sh) * 0x01010101u;
  const uint64_t magic2 = pack2f(kRoundMagic, kRoundMagic);
  uint32_t S = 0;
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const uint32_t inside = (2u * h < nvalid ? 0x00ff00ffu : 0u) | (2u * h + 1u < nvalid ? 0xff00ff00u : 0u);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      if (SV) {
        const uint32_t q4 = codes4<BF16, true>(x[8 * h + i], x[8 * h + 4 + i], low) & inside;
        S = __vsadu4((tb[4 * h + i] >> sh) & shmask, q4) + S;
        ql[4 * h + i] = q4;
        continue;
      }
      const uint32_t q4 = bytes4(quotient2(magnitudes2<BF16>(x[8 * h + i]), low, magic2),
                                 quotient2(magnitudes2<BF16>(x[8 * h + 4 + i]), low, magic2));
      S = __vsadu4((tb[4 * h + i] >> sh) & shmask, q4) + S;
      ql[4 * h + i] = q4;
    }
  }
  return S;
}

// Bytes of one group as distortion_first leaves them -> bit-planes: on return r[k] = bit k of every byte,
// k < 7 code bits, k = 7 signs.
__device__ __forceinline__ void planes_of_bytes(const uint32_t (&tb)[8], uint32_t (&r)[8]) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    r[2 * i] = __byte_perm(tb[i], tb[4 + i], 0x5410);      // byte c = element 8c + 2i
    r[2 * i + 1] = __byte_perm(tb[i], tb[4 + i], 0x7632);  // byte c = element 8c + 2i + 1
  }
  transpose8x32_select(r);
}

// Pass C on one group of a row whose chosen level is plain: codes as bytes (code | sign << 7), transposed into
// bit-planes: on return r[k] = bit k of every byte, k < 7 code bits, k = 7 signs.
template <bool BF16, bool SV = false>
__device__ __forceinline__ void pack_group(const uint32_t (&x)[16], const Level2& lv, uint32_t (&r)[8], uint32_t nvalid = 4u) {
  const uint64_t magic2 = pack2f(kRoundMagic, kRoundMagic);
  uint32_t tb[8];
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const uint32_t inside = (2u * h < nvalid ? 0x00ff00ffu : 0u) | (2u * h + 1u < nvalid ? 0xff00ff00u : 0u);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const uint32_t xa = x[8 * h + i], xb = x[8 * h + 4 + i];
      if (SV) {
        tb[4 * h + i] = codes4<BF16, true>(xa, xb, lv) & inside;
        continue;
      }
      const uint32_t c4 = bytes4(quotient2(magnitudes2<BF16>(xa), lv, magic2), quotient2(magnitudes2<BF16>(xb), lv, magic2));
      tb[4 * h + i] = c4 | (__byte_perm(xa, xb, 0x7351) & 0x80808080u);
    }
  }
  planes_of_bytes(tb, r);
}

// The same steps with the division instruction, for one group held in registers (the one-CTA-per-row kernel).
// (SV: the zeros past the end of a row would get non-zero codes under a negative zero-point, so only the
// first `pairs` registers, the ones inside the row, count.)
template <bool BF16, bool SV = false>
__device__ __forceinline__ uint32_t divide_distortion_regs(const uint32_t (&x)[16], const Level& top, const Level& low, int sh,
                                                           uint32_t pairs = 16u) {
  const uint32_t shmask = (0xffffu >> sh) * 0x10001u;
  uint32_t S = 0;
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    if (SV && static_cast<uint32_t>(i) >= pairs) continue;
    const uint32_t a = (codes2_divide<BF16, SV>(x[i], top) >> sh) & shmask;
    const uint32_t q = codes2_divide<BF16, SV>(x[i], low);
    const uint32_t d = max_s16x2(a, q) - min_s16x2(a, q);
    S += (d & 0xffffu) + (d >> 16);
  }
  return S;
}

struct Planes8 {
  uint32_t v[8];
};
template <bool BF16, bool SV = false>
__device__ __forceinline__ void divide_pack_regs(const uint32_t (&x)[16], const Level& lv, uint32_t (&r)[8]) {
#pragma unroll
  for (int k = 0; k < 8; ++k) r[k] = 0u;  // r[k] bit e = bit k of the byte (code | sign << 7; SV: the 8-bit code) of element e
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    // elements 2i (byte 0) and 2i + 1 (byte 2)
    const uint32_t b2 = codes2_divide<BF16, SV>(x[i], lv) | (SV ? 0u : ((x[i] >> 8) & 0x00800080u));
#pragma unroll
    for (int k = 0; k < 8; ++k) r[k] |= (((b2 >> k) & 1u) << (2 * i)) | (((b2 >> (16 + k)) & 1u) << (2 * i + 1));
  }
}

// The same two steps for rows that need the division instruction, written as loops over the parked
// row's words (xw: the row as 32-bit words) so that they take little room in the instruction stream.
__device__ __forceinline__ uint32_t park_index(uint32_t nt, uint32_t u, uint32_t j);
// (SV: only the first `pairs` words, the ones inside the row, count: see divide_distortion_regs.)
template <bool BF16, bool SV = false>
__device__ __noinline__ uint32_t rolled_distortion(const uint32_t* xw, uint32_t nt, uint32_t u, Level top, Level low, int sh,
                                                   uint32_t pairs = 16u) {
  const uint32_t shmask = (0xffffu >> sh) * 0x10001u;
  uint32_t S = 0;
#pragma unroll 1
  for (uint32_t i = 0; i < (SV ? pairs : 16u); ++i) {
    const uint32_t x = xw[4u * park_index(nt, u, i >> 2) + (i & 3u)];
    const uint32_t a = (codes2_divide<BF16, SV>(x, top) >> sh) & shmask;
    const uint32_t q = codes2_divide<BF16, SV>(x, low);
    const uint32_t d = max_s16x2(a, q) - min_s16x2(a, q);
    S += (d & 0xffffu) + (d >> 16);
  }
  return S;
}
template <bool BF16, bool SV = false>
__device__ __noinline__ Planes8 rolled_pack(const uint32_t* xw, uint32_t nt, uint32_t u, Level lv, uint32_t pairs = 16u) {
  uint32_t r[8] = {0, 0, 0, 0, 0, 0, 0, 0};  // r[k] bit e = bit k of the byte (code | sign << 7; SV: the 8-bit code) of element e
#pragma unroll 1
  for (uint32_t i = 0; i < (SV ? pairs : 16u); ++i) {
    const uint32_t x = xw[4u * park_index(nt, u, i >> 2) + (i & 3u)];
    // elements 2i (byte 0) and 2i + 1 (byte 2)
    const uint32_t b2 = codes2_divide<BF16, SV>(x, lv) | (SV ? 0u : ((x >> 8) & 0x00800080u));
#pragma unroll
    for (int k = 0; k < 8; ++k) r[k] |= (((b2 >> k) & 1u) << (2u * i)) | (((b2 >> (16 + k)) & 1u) << (2u * i + 1u));
  }
  Planes8 out;
#pragma unroll
  for (int k = 0; k < 8; ++k) out.v[k] = r[k];
  return out;
}

// Shared-memory index (in 16-byte chunks) of chunk j of group u inside a parked row of nt groups: a group's
// four chunks stay together, rotated so that the 16-byte accesses of neighbouring threads fall into
// different banks.  (Keeping the chunks with the same j side by side instead measured 8 % slower while the
// copies bypassed L1, and no faster than this since they do not.)
__device__ __forceinline__ uint32_t park_index(uint32_t /*nt*/, uint32_t u, uint32_t j) { return 4u * u + ((j + (u >> 1)) & 3u); }

// Number of 16-byte chunks of group u that lie inside the row (4, fewer in the last group, 0 beyond it).
// Recomputed where it is needed: a value kept alive across the whole row loop costs a register there.
__device__ __forceinline__ uint32_t group_chunks(const EncodeParams& p, uint32_t u) {
  return 4u * u < p.chunks ? min(p.chunks - 4u * u, 4u) : 0u;
}

// Asynchronous copy of the 64 bytes of group u of row `tile` into parked row `slot` (chunks
// j >= nvalid lie past the end of the row and are not copied).
__device__ __forceinline__ void fetch_group(const EncodeParams& p, uint4* xpark, uint32_t tile, uint32_t slot, uint32_t u,
                                            uint32_t nvalid) {
  const uint4* xrow = reinterpret_cast<const uint4*>(p.x + static_cast<size_t>(tile) * p.hidden);
  uint4* xp = xpark + slot * (p.park_stride / 16u);
#pragma unroll
  for (uint32_t j = 0; j < 4; ++j) {
    if (j < nvalid) cp_async16(&xp[park_index(p.compute_threads, u, j)], &xrow[4u * u + j]);
  }
  cp_async_commit();
}

// The CSR entries (column << 16 | original pattern) of the elements of one group that `bm` flags, in
// ascending column order, from the group's 64 bytes as they stand in the input (v[j] = chunk j): f(entry) is
// called once per flagged element.  All 32 positions are visited under a predicate: no data-dependent loads.
template <typename F>
__device__ __forceinline__ void for_each_flagged(uint32_t bm, const uint4 (&v)[4], uint32_t col0, F&& f) {
#pragma unroll
  for (uint32_t j = 0; j < 4; ++j) {
    const uint32_t w[4] = {v[j].x, v[j].y, v[j].z, v[j].w};
#pragma unroll
    for (uint32_t i = 0; i < 4; ++i) {
      const uint32_t e = 8u * j + 2u * i;
      if ((bm >> e) & 1u) f(((col0 + e) << 16) | (w[i] & 0xffffu));
      if ((bm >> (e + 1u)) & 1u) f(((col0 + e + 1u) << 16) | (w[i] >> 16));
    }
  }
}

// The b* plane words of one group, in blob order (plane 0 = sign, plane 1 + k = code bit k), to dst.
// SV: plane k = code bit k, no sign plane.
template <bool SV = false>
__device__ __forceinline__ void store_planes(uint32_t* dst, const uint32_t (&r)[8], int bstar, bool vec) {
  if (SV) {
    if (vec && bstar == 8) {
      reinterpret_cast<uint4*>(dst)[0] = make_uint4(r[0], r[1], r[2], r[3]);
      reinterpret_cast<uint4*>(dst)[1] = make_uint4(r[4], r[5], r[6], r[7]);
    } else if (vec && bstar == 4) {
      reinterpret_cast<uint4*>(dst)[0] = make_uint4(r[0], r[1], r[2], r[3]);
    } else {
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        if (q < bstar) dst[q] = r[q];
      }
    }
    return;
  }
  if (vec && bstar == 8) {
    reinterpret_cast<uint4*>(dst)[0] = make_uint4(r[7], r[0], r[1], r[2]);
    reinterpret_cast<uint4*>(dst)[1] = make_uint4(r[3], r[4], r[5], r[6]);
  } else if (vec && bstar == 4) {
    reinterpret_cast<uint4*>(dst)[0] = make_uint4(r[7], r[0], r[1], r[2]);
  } else {
    dst[0] = r[7];
#pragma unroll
    for (int q = 0; q < 7; ++q) {
      if (q < bstar - 1) dst[1 + q] = r[q];
    }
  }
}

// The row's min / max patterns, outlier total and per-warp outlier offsets from the per-warp partial
// results, and the AIQ parameters of every candidate: run by one full warp, lane i takes candidate i.
// Returns (in every lane) 1 when some level needs the division instruction.
template <int NW>  // the most warps that contribute
struct RowPartials {
  uint32_t warp_min[NW], warp_max[NW], warp_cnt[NW];  // warp_cnt becomes an exclusive scan
};
template <bool BF16, int NW, bool SV = false>
__device__ __forceinline__ uint32_t row_levels(const EncodeParams& p, RowPartials<NW>& part, uint32_t nwarps, uint32_t lane,
                                               Level* lv_out, int* S_out, uint32_t* row_cnt) {
  using E = Elem<BF16>;
  const uint32_t pmin = __reduce_min_sync(kFull, lane < nwarps ? part.warp_min[lane] : 0xffffu);
  const uint32_t pmax = __reduce_max_sync(kFull, lane < nwarps ? part.warp_max[lane] : 0u);
  const uint32_t wc = lane < nwarps ? part.warp_cnt[lane] : 0u;
  uint32_t incl = wc;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const uint32_t n = __shfl_up_sync(kFull, incl, d);
    if (lane >= static_cast<uint32_t>(d)) incl += n;
  }
  if (lane < nwarps) part.warp_cnt[lane] = incl - wc;
  const uint32_t total = __shfl_sync(kFull, incl, 31);
  // SV: the partial results are order keys of signed values
  const int b = p.bits[min(lane, static_cast<uint32_t>(p.n_bits - 1))];
  bool plain = false;
  const Level lv = SV ? make_level_signed(E::pattern_f32(pattern_of_key(pmin)), E::pattern_f32(pattern_of_key(pmax)), b, &plain)
                      : make_level(E::pattern_f32(pmin), E::pattern_f32(pmax), b, &plain);
  if (lane < static_cast<uint32_t>(p.n_bits)) {
    lv_out[lane] = lv;
    S_out[lane] = 0;
  }
  if (lane == 0) *row_cnt = total;
  return __all_sync(kFull, plain) ? 0u : 1u;
}

// The limit on device-side waits: the workspace's setting, else the built-in one.
__device__ __forceinline__ uint32_t lookback_limit(const EncodeParams& p) {
  const uint32_t set = *reinterpret_cast<volatile const uint32_t*>(&p.ws->poll_limit);
  return set != 0u ? set : kLookbackPollLimit;
}

__device__ __forceinline__ unsigned long long pack_desc(uint32_t tag, uint32_t value) {
  return (static_cast<unsigned long long>(tag) << 32) | value;
}

// Decoupled look-back over the tile descriptors.
// Tile t owns two adjacent descriptors, desc[2t] for plane words and desc[2t + 1] for outliers, each
// (generation * 4 + flag) << 32 | payload: an AGGREGATE payload is the tile's own size, a PREFIX
// payload the inclusive prefix sum up to and including the tile.  Both are read in the same round
// trip; a tile counts as published once both carry the same flag of the current generation.
__device__ __forceinline__ void publish(const EncodeParams& p, uint32_t tag, uint32_t tile, uint32_t w, uint32_t o) {
  st_relaxed_u64(p.desc + 2 * static_cast<size_t>(tile), pack_desc(tag, w));
  st_relaxed_u64(p.desc + 2 * static_cast<size_t>(tile) + 1, pack_desc(tag, o));
}

__device__ __forceinline__ void publish_aggregate(const EncodeParams& p, uint32_t gen4, uint32_t tile, uint32_t agg_w,
                                                  uint32_t agg_o) {
  if (tile > 0) publish(p, gen4 | kFlagAggregate, tile, agg_w, agg_o);
}

// State of a tile from its two descriptors: 0 = not (consistently) published yet, else the common flag.
__device__ __forceinline__ uint32_t tile_state(uint32_t gen4, unsigned long long vw, unsigned long long vo) {
  const uint32_t tw = static_cast<uint32_t>(vw >> 32), to = static_cast<uint32_t>(vo >> 32);
  const uint32_t fw = ((tw & ~3u) == gen4) ? (tw & 3u) : 0u, fo = ((to & ~3u) == gen4) ? (to & 3u) : 0u;
  if (fw == kFlagAbort || fo == kFlagAbort) return kFlagAbort;
  return fw == fo ? fw : 0u;
}

// Run by one full warp for its tile, after publish_aggregate: walk back to the nearest published
// prefix, then publish this tile's own.
// Returns TSQ_OK, TSQ_ERR_TIMEOUT (gave up) or -1 when a predecessor has aborted.
// DEPTH = descriptor pairs each lane reads per step (32 * DEPTH tiles per round trip).  The one-CTA-per-row
// kernel, whose rows all finish at about the same time, looks back 256 tiles at once; the pipelined
// kernel, where the nearest finished prefix is rarely more than a few dozen tiles away and the look-back
// runs in a lone warp that issues slowly, takes 32 (measured: 6 % faster at hidden 8192 and 20 % at
// 1024 than with 256).
template <int DEPTH>
__device__ int resolve_prefix(const EncodeParams& p, uint32_t gen4, uint32_t tile, uint32_t agg_w, uint32_t agg_o,
                              uint32_t lane, uint32_t* excl_w, uint32_t* excl_o, uint32_t poll_limit) {
  uint32_t base_w = 0, base_o = 0;  // prefix found at the end of the walk
  uint32_t part_w = 0, part_o = 0;  // this lane's share of the aggregates walked over
  if (tile > 0) {
    int pos = static_cast<int>(tile) - 1;  // nearest tile not yet accounted for
    uint32_t polls = 0;
    bool done = false;
    while (!done) {
      unsigned long long vw[DEPTH], vo[DEPTH];
#pragma unroll
      for (int k = 0; k < DEPTH; ++k) {
        const int j = pos - (32 * k + static_cast<int>(lane));
        // before tile 0: prefix 0
        vw[k] = vo[k] = pack_desc(gen4 | kFlagPrefix, 0u);
        if (j >= 0) ld_relaxed_u64x2(p.desc + 2 * static_cast<size_t>(j), vw[k], vo[k]);
      }
      int consumed = 32 * DEPTH;
      bool stopped = false;
      int verdict = TSQ_OK;
#pragma unroll
      for (int k = 0; k < DEPTH; ++k) {
        if (stopped) continue;
        // the usual window: 32 aggregates
        const uint32_t agg_tag = gen4 | kFlagAggregate;
        if (__all_sync(kFull, static_cast<uint32_t>(vw[k] >> 32) == agg_tag && static_cast<uint32_t>(vo[k] >> 32) == agg_tag)) {
          part_w += static_cast<uint32_t>(vw[k]);
          part_o += static_cast<uint32_t>(vo[k]);
          continue;
        }
        const uint32_t state = tile_state(gen4, vw[k], vo[k]);
        const uint32_t stop = __ballot_sync(kFull, state != kFlagAggregate);
        const uint32_t first = stop ? static_cast<uint32_t>(__ffs(stop) - 1) : 32u;
        if (lane < first) {
          part_w += static_cast<uint32_t>(vw[k]);
          part_o += static_cast<uint32_t>(vo[k]);
        }
        if (stop == 0u) continue;
        stopped = true;
        const uint32_t first_state = __shfl_sync(kFull, state, first);
        if (first_state == kFlagAbort) {
          verdict = -1;
        } else if (first_state == kFlagPrefix) {
          base_w = __shfl_sync(kFull, static_cast<uint32_t>(vw[k]), first);
          base_o = __shfl_sync(kFull, static_cast<uint32_t>(vo[k]), first);
          done = true;
        } else {  // not published yet: keep what was walked over, poll again from there
          consumed = 32 * k + static_cast<int>(first);
        }
      }
      if (verdict != TSQ_OK) return verdict;
      if (!done) {
        pos -= consumed;
        if (consumed == 0) {
          // tile `pos` has published nothing yet: watch its two descriptors alone until it has
          for (;;) {
            uint32_t state = 0u;
            if (lane == 0) {
              unsigned long long w0, w1;
              ld_relaxed_u64x2(p.desc + 2 * static_cast<size_t>(pos), w0, w1);
              state = tile_state(gen4, w0, w1);
            }
            if (__shfl_sync(kFull, state, 0) != 0u) break;
            if (++polls > poll_limit) return TSQ_ERR_TIMEOUT;
            __nanosleep(polls < 32u ? 200u : 1000u);
          }
        }
      }
    }
    base_w += __reduce_add_sync(kFull, part_w);
    base_o += __reduce_add_sync(kFull, part_o);
  }
  if (lane == 0) publish(p, gen4 | kFlagPrefix, tile, base_w + agg_w, base_o + agg_o);
  *excl_w = base_w;
  *excl_o = base_o;
  return TSQ_OK;
}

__device__ void write_header(const EncodeParams& p, unsigned long long total_words, unsigned long long total_outliers) {
  BlobHeader* h = reinterpret_cast<BlobHeader*>(p.blob);
  h->magic = kMagic;
  h->version = kVersion;
  h->dtype = p.dtype;
  h->hidden = p.hidden;
  h->tokens = p.tokens;
  h->n_bits = static_cast<uint32_t>(p.n_bits);
#pragma unroll
  for (int i = 0; i < 7; ++i) h->bits[i] = (i < p.n_bits) ? static_cast<uint8_t>(p.bits[i]) : 0;
  h->bits[7] = static_cast<uint8_t>(p.variant);  // at most seven candidates: the last entry carries the variant
  h->tau = p.tau;
  h->delta = p.delta;
  h->total_words = total_words;
  h->total_outliers = total_outliers;
  h->outlier_capacity = static_cast<uint32_t>(p.lay.outlier_capacity);
}

// The CTA that finishes last publishes the totals and the status, and re-arms the workspace.
__device__ void finish_call(const EncodeParams& p, uint32_t gen4) {
  __threadfence();
  const uint32_t prev = atomicAdd(&p.ws->done, 1u);
  if (prev != gridDim.x - 1u) return;
  __threadfence();
  const uint32_t e = atomicExch(&p.ws->err, 0u);
  // totals = the last tile's inclusive prefixes, if it got that far
  unsigned long long tw = 0ull, to = 0ull;
  if (p.tokens != 0u) {
    const unsigned long long dw = ld_relaxed_u64(p.desc + 2 * static_cast<size_t>(p.tokens - 1u));
    const unsigned long long dout = ld_relaxed_u64(p.desc + 2 * static_cast<size_t>(p.tokens - 1u) + 1);
    if (tile_state(gen4, dw, dout) == kFlagPrefix) {
      tw = static_cast<uint32_t>(dw);
      to = static_cast<uint32_t>(dout);
    }
  }
  write_header(p, tw, to);
  reinterpret_cast<BlobHeader*>(p.blob)->status = e;
  if (p.tokens == 0u) {  // no row writes the leading zeros of the two prefix-sum sections
    reinterpret_cast<uint32_t*>(p.blob + p.lay.off_word_off)[0] = 0u;
    reinterpret_cast<uint32_t*>(p.blob + p.lay.off_out_ptr)[0] = 0u;
  }
  if (e != 0u) atomicCAS(&p.ws->enc_status, 0u, e);
  uint32_t g = (gen4 >> 2);
  if (g >= kGenWrap) {
    // generation counter about to wrap: wipe the descriptors so that old tags cannot alias
    const uint32_t n = p.ws->desc_capacity;
    for (uint32_t i = 0; i < 2u * n; ++i) p.desc[i] = 0ull;
    g = 0u;
  }
  p.ws->ticket = 0u;
  p.ws->done = 0u;
  p.ws->gen = g;
}

// The per-token fields of the blob, written by one thread.
__device__ __forceinline__ void write_token_fields(const EncodeParams& p, uint32_t tile, int bstar, float scale, int zp,
                                                   uint32_t word_end, uint32_t out_end) {
  reinterpret_cast<uint8_t*>(p.blob + p.lay.off_bits)[tile] = static_cast<uint8_t>(bstar);
  reinterpret_cast<float*>(p.blob + p.lay.off_scale)[tile] = scale;
  reinterpret_cast<int32_t*>(p.blob + p.lay.off_zp)[tile] = zp;
  uint32_t* o_word_off = reinterpret_cast<uint32_t*>(p.blob + p.lay.off_word_off);
  uint32_t* o_out_ptr = reinterpret_cast<uint32_t*>(p.blob + p.lay.off_out_ptr);
  if (tile == 0) {
    o_word_off[0] = 0;
    o_out_ptr[0] = 0;
  }
  o_word_off[tile + 1] = word_end;
  o_out_ptr[tile + 1] = out_end;
}

// =====================================================================================================
// encode_rows_kernel: one CTA per row, everything in order.
// =====================================================================================================

struct RowShared {
  Level lv[kMaxCand];  // lv[i]: AIQ parameters of candidate bits[i]
  int S[kMaxCand];     // distortion sum of candidate i against the top level
  RowPartials<32> part;
  uint32_t tile;
  uint32_t divide;     // some level of the row needs the division instruction
  uint32_t row_cnt;    // outliers of the row
  uint32_t word_off, out_base;
  uint32_t status;     // TSQ_OK, or why the row is not written
};

// MAXT: the largest CTA the instance is launched with (rows of up to 8192 elements get the 256-thread instance,
// which may use four times the registers of the 1024-thread one).  SV: the signed-values variant.
template <bool BF16, int UPT, int MAXT, bool SV>
__global__ void __launch_bounds__(MAXT, MAXT == 256 ? 2 : 1) encode_rows_kernel(const EncodeParams p) {
  using E = Elem<BF16>;
  __shared__ RowShared sh;
  const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5, nwarps = blockDim.x >> 5;
  const uint32_t gen4 = (*reinterpret_cast<volatile const uint32_t*>(&p.ws->gen) + 1u) << 2;

  if (tid == 0) {
    // a call whose rows all get a CTA at once needs no ticket: every CTA is running, so row = CTA index is safe
    sh.tile = p.direct_tiles != 0u ? blockIdx.x : atomicAdd(&p.ws->ticket, 1u);
    sh.status = TSQ_OK;
  }
  __syncthreads();
  const uint32_t tile = sh.tile;

  if (tile < p.tokens) {
    // ---- the row, 64 bytes per group, straight into registers; thread t owns groups UPT * t + k ----
    uint32_t x[UPT][16];
    uint32_t nvalid[UPT];
    const uint4* xrow = reinterpret_cast<const uint4*>(p.x + static_cast<size_t>(tile) * p.hidden);
#pragma unroll
    for (int k = 0; k < UPT; ++k) {
      const uint32_t u = UPT * tid + k;
      nvalid[k] = 4u * u < p.chunks ? min(p.chunks - 4u * u, 4u) : 0u;
#pragma unroll
      for (uint32_t j = 0; j < 4; ++j) {
        const uint4 c = j < nvalid[k] ? xrow[4u * u + j] : make_uint4(0u, 0u, 0u, 0u);
        x[k][4 * j + 0] = c.x;
        x[k][4 * j + 1] = c.y;
        x[k][4 * j + 2] = c.z;
        x[k][4 * j + 3] = c.w;
      }
    }

    // ---- pass A: threshold split, min / max of the inlier magnitudes, outlier counts ----
    const uint32_t thr2 = p.thr16 * 0x10001u;
    uint32_t mn2 = E::kInfPattern * 0x10001u, mx2 = 0u;
    uint32_t bitmap[UPT];
    uint32_t cnt = 0u;
#pragma unroll
    for (int k = 0; k < UPT; ++k) {
      bitmap[k] = split_group<BF16>(x[k], nvalid[k], thr2, mn2, mx2);
      cnt += __popc(bitmap[k]);
    }
    if (SV) {
      // min / max of the signed values of T_below instead (outlier slots are +0 by now): as order keys
      mn2 = 0xffffffffu;
      mx2 = 0u;
#pragma unroll
      for (int k = 0; k < UPT; ++k) {
#pragma unroll
        for (uint32_t i = 0; i < 16; ++i) {
          if ((i >> 2) < nvalid[k]) {
            const uint32_t key2 = order_keys2(x[k][i]);
            mn2 = __vminu2(mn2, key2);
            mx2 = __vmaxu2(mx2, key2);
          }
        }
      }
    }
    {
      const uint32_t mnv = __reduce_min_sync(kFull, min(mn2 & 0xffffu, mn2 >> 16));
      const uint32_t mxv = __reduce_max_sync(kFull, max(mx2 & 0xffffu, mx2 >> 16));
      const uint32_t wcnt = __reduce_add_sync(kFull, cnt);
      if (lane == 0) {
        sh.part.warp_min[warp] = mnv;
        sh.part.warp_max[warp] = mxv;
        sh.part.warp_cnt[warp] = wcnt;
      }
    }
    __syncthreads();

    // ---- AIQ parameters of every candidate level (lane i of warp 0 takes candidate i) ----
    const int bmax = p.bits[p.n_bits - 1];
    if (warp == 0) {
      const uint32_t divide = row_levels<BF16, 32, SV>(p, sh.part, nwarps, lane, sh.lv, sh.S, &sh.row_cnt);
      if (lane == 0) sh.divide = divide;
    }
    __syncthreads();
    const bool divide = sh.divide != 0u;

    // ---- Algorithm 1: descend the candidate list while the distortion stays within tolerance ----
    const Level top = sh.lv[p.n_bits - 1];
    Level best = top;
    int bstar = bmax;
    for (int ci = p.n_bits - 2; ci >= 0; --ci) {
      const Level low = sh.lv[ci];
      const int shn = bmax - p.bits[ci];
      uint32_t S = 0;
#pragma unroll
      for (int k = 0; k < UPT; ++k) {
        if (divide) {
          S += divide_distortion_regs<BF16, SV>(x[k], top, low, shn, 4u * nvalid[k]);
        } else {
          S += distortion_group<BF16, SV>(x[k], make_level2(top), make_level2(low), shn, nvalid[k]);
        }
      }
      S = __reduce_add_sync(kFull, S);
      if (lane == 0 && S != 0u) atomicAdd(&sh.S[ci], static_cast<int>(S));
      __syncthreads();
      if (sh.S[ci] > p.s_max) break;  // delta > Delta: keep the last level that passed
      bstar = p.bits[ci];
      best = low;
    }
    const uint32_t row_cnt = sh.row_cnt;
    const uint32_t agg_w = static_cast<uint32_t>(bstar) * p.lay.wpp;

    // ---- this row's sizes are known: let the rows behind it see them, then pack ----
    if (tid == 0) publish_aggregate(p, gen4, tile, agg_w, row_cnt);
    uint32_t r[UPT][8];
#pragma unroll
    for (int k = 0; k < UPT; ++k) {
      if (divide) {
        divide_pack_regs<BF16, SV>(x[k], best, r[k]);
        if (SV && nvalid[k] < 4u) {  // pad bits stay 0: the zeros past the end of the row got the code of the value 0
          const uint32_t inside = (1u << (8u * nvalid[k])) - 1u;
#pragma unroll
          for (int q = 0; q < 8; ++q) r[k][q] &= inside;
        }
      } else {
        pack_group<BF16, SV>(x[k], make_level2(best), r[k], nvalid[k]);
      }
    }

    // ---- placement: exclusive prefix sums over the tokens before this one ----
    if (warp == 0) {
      uint32_t word_off = 0, out_base = 0;
      const int st = resolve_prefix<8>(p, gen4, tile, agg_w, row_cnt, lane, &word_off, &out_base, lookback_limit(p));
      if (lane == 0) {
        sh.word_off = word_off;
        sh.out_base = out_base;
        if (st != TSQ_OK) {
          publish(p, gen4 | kFlagAbort, tile, 0u, 0u);
          sh.status = st < 0 ? 0xffffffffu : static_cast<uint32_t>(st);
          if (st > 0) atomicCAS(&p.ws->err, 0u, static_cast<uint32_t>(st));
        }
      }
    }
    __syncthreads();

    if (sh.status == TSQ_OK) {
      const uint32_t word_off = sh.word_off, out_base = sh.out_base;
      // ---- plane words: group u owns words u * b* .. u * b* + b* - 1 ----
      uint32_t* wrow = reinterpret_cast<uint32_t*>(p.blob + p.lay.off_words) + word_off;
#pragma unroll
      for (int k = 0; k < UPT; ++k) {
        const uint32_t u = UPT * tid + k;
        if (u < p.units) store_planes<SV>(wrow + static_cast<size_t>(u) * bstar, r[k], bstar, p.vec_store != 0u);
      }
      if (tid == 0) write_token_fields(p, tile, bstar, best.s, best.zp, word_off + agg_w, out_base + row_cnt);
      // ---- CSR entries of T_above: ascending columns, original patterns (read again from the input) ----
      if (__ballot_sync(kFull, cnt != 0u) != 0u) {
        uint32_t incl = cnt;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
          const uint32_t n = __shfl_up_sync(kFull, incl, d);
          if (lane >= static_cast<uint32_t>(d)) incl += n;
        }
        if (cnt != 0u) {
          uint32_t* o_outl = reinterpret_cast<uint32_t*>(p.blob + p.lay.off_outl);
          const uint16_t* x16 = p.x + static_cast<size_t>(tile) * p.hidden;
          unsigned long long at = static_cast<unsigned long long>(out_base) + sh.part.warp_cnt[warp] + (incl - cnt);
          bool overflow = false;
#pragma unroll
          for (int k = 0; k < UPT; ++k) {
            uint32_t bm = bitmap[k];
            const uint32_t u = UPT * tid + k;
            while (bm != 0u) {
              const uint32_t e = 32u * u + static_cast<uint32_t>(__ffs(bm) - 1);
              bm &= bm - 1u;
              if (at < p.lay.outlier_capacity) {
                o_outl[at] = (e << 16) | x16[e];
              } else {
                overflow = true;
              }
              ++at;
            }
          }
          if (overflow) atomicCAS(&p.ws->err, 0u, static_cast<uint32_t>(TSQ_ERR_OUTLIER_OVERFLOW));
        }
      }
    }
  }

  __syncthreads();
  if (tid == 0) finish_call(p, gen4);
}

// =====================================================================================================
// encode_pipe_kernel: persistent CTAs, rows in several stages at once.
// =====================================================================================================
// Threads: `compute` threads (one per 32-element group of a row, a multiple of 32), then the levels
// warp, then the placement warp.  Row n of a CTA (n = 0, 1, ... in the order it takes them):
//   compute warps, iteration n - 1  asynchronous copies of the row into xpark[n % 3], 64 bytes per thread
//   compute warps, iteration n      pass A on the thread's own 64 bytes, thresholded values written back in
//                                   place; per-warp partial results in meta[n % kMetaRing]
//   levels warp                     meta[..].lv = AIQ parameters of every candidate (after a_ready > n)
//   compute warps, iteration n + 1  passes B and C from the parked copy (after lv_ready > n), planes
//                                   into planes[n % ring], CSR entries into csr[n % ring]
//   placement warp                  offsets by look-back, bulk store of the planes, token fields, CSR
//                                   entries (after packed > n); then placed = n + 1 frees the slots.
// Each thread copies, thresholds and re-reads only its own group, so the parked rows need no barrier.  All counters
// only grow; every wait on them is bounded and raises `abort`.

// Rows a CTA may hold between packing and placement: p.ring (2 .. kMaxRing) slots of planes and CSR entries,
// as many as fit beside the parked rows.  Placement waits for the rows before it, so a deep ring is what
// keeps the compute warps busy while a slow predecessor (a row whose descent goes on) holds everybody up.
constexpr int kMetaRing = kMaxRing + 2;  // row records: one row in pass A and one being packed on top of those

struct RowMeta {
  Level lv[kMaxCand];
  int S[kMaxCand];
  RowPartials<(kPipeMaxThreads - 64) / 32> part;
  uint32_t tile, row_cnt, divide;
  uint32_t bstar, agg_w;
  float scale;
  int zp;
  uint32_t heavy;  // 1: the side buffer holds the row's outlier bitmaps (more outliers than a list holds)
};

struct PipeShared {
  RowMeta meta[kMetaRing];
  volatile uint32_t a_ready;   // rows whose pass A results are in their record
  volatile uint32_t lv_ready;  // rows whose levels are computed
  volatile uint32_t packed;    // rows packed and parked
  volatile uint32_t placed;    // rows placed
  volatile uint32_t finished;  // the compute warps are done: a_ready and packed are final
  volatile uint32_t abort;     // a wait inside the CTA ran out
  volatile uint32_t stop[2];   // abort as thread 0 saw it before the iteration's barrier, by iteration parity: what the
                               // compute threads act on, so that all of them leave the row loop in the same iteration
  uint32_t wait_limit;         // polls before a handshake gives up
  uint32_t next_tile[2];       // ticket of the row after the current one, by iteration parity
  // Rows with more outliers than a ring slot's list holds: the compute threads leave the groups' bitmaps in a side
  // buffer, the placement warp posts the row's CSR offset there once it is resolved, and the compute threads write
  // the entries themselves, all at once, at the top of a later iteration.  (One buffer: a second one would cost
  // the ring a slot at hidden 8192.  A row that finds it taken leaves its bitmaps in the list instead.)
  uint32_t heavy_bm[kPipeMaxThreads - 64];
  uint32_t heavy_wcnt[(kPipeMaxThreads - 64) / 32];  // exclusive scan of the warps' outlier counts
  uint32_t heavy_tile;
  volatile uint32_t heavy_base;      // out_ptr[tile], from the placement warp
  volatile uint32_t heavy_posted;    // such rows whose offset has been posted
  volatile uint32_t heavy_seen[2];   // heavy_posted as thread 0 saw it before the iteration's barrier, by iteration parity
};

__device__ __forceinline__ void compute_barrier(uint32_t nthreads) {
  asm volatile("bar.sync 1, %0;" ::"r"(nthreads) : "memory");
}

// Wait until *counter > n.  Returns false when the wait is to be given up: `finished` is set and the
// counter will not grow any more, or the CTA aborted, or the limit ran out (which raises abort).
__device__ __forceinline__ bool wait_beyond(volatile uint32_t* counter, uint32_t n, PipeShared& sh, bool may_finish,
                                            uint32_t nap_ns) {
  for (uint32_t polls = 0;; ++polls) {
    if (*counter > n) return true;
    if (sh.abort != 0u) return false;
    if (may_finish && sh.finished != 0u) return *counter > n;
    if (polls > sh.wait_limit) {
      sh.abort = 1u;
      return false;
    }
    __nanosleep(nap_ns);
  }
}

// FULL: every compute thread owns a whole 32-element group (hidden is a multiple of 1024), so none of the
// checks for short or missing groups is needed.
// SV: the signed-values variant.
template <bool BF16, bool FULL, int MAXT, int MINB, bool SV>
__global__ void __launch_bounds__(MAXT, MINB) encode_pipe_kernel(const EncodeParams p) {
  using E = Elem<BF16>;
  extern __shared__ __align__(128) unsigned char smem_dyn[];
  __shared__ PipeShared sh;
  const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
  const uint32_t nt = p.compute_threads, nwarps = nt >> 5;
  const uint32_t gen4 = (*reinterpret_cast<volatile const uint32_t*>(&p.ws->gen) + 1u) << 2;
  uint4* const xpark = reinterpret_cast<uint4*>(smem_dyn);
  uint32_t* const planes = reinterpret_cast<uint32_t*>(smem_dyn + 3u * p.park_stride);
  uint32_t* const csr = reinterpret_cast<uint32_t*>(smem_dyn + 3u * p.park_stride + p.ring * p.planes_stride);  // p.ring lists of p.csr_cap entries

  if (tid == 0) {
    sh.a_ready = 0u;
    sh.lv_ready = 0u;
    sh.packed = 0u;
    sh.placed = 0u;
    sh.finished = 0u;
    sh.abort = 0u;
    sh.stop[0] = sh.stop[1] = 0u;
    sh.heavy_posted = 0u;
    sh.heavy_seen[0] = sh.heavy_seen[1] = 0u;
    {
      const uint32_t lim = lookback_limit(p);
      sh.wait_limit = lim > 0xffffffffu / kHandshakeFactor ? 0xffffffffu : lim * kHandshakeFactor;
    }
    sh.next_tile[0] = atomicAdd(&p.ws->ticket, 1u);
  }
  __syncthreads();

  if (tid < nt) {
    // ================================ compute warps ================================
    const uint32_t u = tid;  // this thread's group in every row
    uint32_t tile_cur = sh.next_tile[0];
    bool have_prev = false;  // row n_a - 1 has been through pass A and is not packed yet
    uint32_t n_a = 0u;       // rows of this CTA that finished pass A; n_a - have_prev of them are packed
    uint32_t bitmap_prev = 0u, cnt_prev = 0u, first_prev = 0u;  // outliers of the thread's group in row n_a - 1
    uint32_t slot = 0u;      // ring slot of the next row to be packed: (rows packed so far) mod p.ring
    uint32_t heavy_filled = 0u, heavy_done = 0u;  // rows put into / written out of the side buffer (the same in every thread)
    // The CSR entries of the row in the side buffer, to their place in the blob: every thread takes its own group.
    const auto emit_heavy = [&]() {
      const uint32_t bm = sh.heavy_bm[u];
      const uint32_t wbase = sh.heavy_wcnt[warp];
      const uint32_t tile_h = sh.heavy_tile;
      const uint32_t base = sh.heavy_base;
      const uint32_t cnt = __popc(bm);
      uint32_t incl = cnt;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const uint32_t v = __shfl_up_sync(kFull, incl, d);
        if (lane >= static_cast<uint32_t>(d)) incl += v;
      }
      if (bm != 0u) {
        unsigned long long at = static_cast<unsigned long long>(base) + wbase + (incl - cnt);
        const uint4* g = reinterpret_cast<const uint4*>(p.x + static_cast<size_t>(tile_h) * p.hidden) + 4u * u;
        const uint32_t nv = FULL ? 4u : group_chunks(p, u);
        uint4 v[4];
#pragma unroll
        for (uint32_t j = 0; j < 4; ++j) v[j] = j < nv ? g[j] : make_uint4(0u, 0u, 0u, 0u);
        uint32_t* o_outl = reinterpret_cast<uint32_t*>(p.blob + p.lay.off_outl);
        bool overflow = false;
        for_each_flagged(bm, v, 32u * u, [&](uint32_t entry) {
          if (at < p.lay.outlier_capacity) {
            o_outl[at] = entry;
          } else {
            overflow = true;
          }
          ++at;
        });
        if (overflow) atomicCAS(&p.ws->err, 0u, static_cast<uint32_t>(TSQ_ERR_OUTLIER_OVERFLOW));
      }
    };
    if (tile_cur < p.tokens) fetch_group(p, xpark, tile_cur, 0u, u, FULL ? 4u : group_chunks(p, u));
    // thread 0: the ticket of the row after tile_cur, asked for a whole iteration before it is needed
    // (the round trip of the atomic is longer than pass A)
    uint32_t ticket_ahead = 0xffffffffu;
    if (tid == 0 && tile_cur < p.tokens) ticket_ahead = atomicAdd(&p.ws->ticket, 1u);

    for (uint32_t it = 0u;; ++it) {
      const bool have_cur = tile_cur < p.tokens;
      if (!have_cur && !have_prev) break;
      uint32_t bitmap_cur = 0u, cnt_cur = 0u, first_cur = 0u;
      if (have_cur) {
        // ---- pass A of row n_a: threshold split in registers, park the row, per-warp partial results ----
        RowMeta& m = sh.meta[n_a % kMetaRing];
        const uint32_t nvalid = FULL ? 4u : group_chunks(p, u);
        uint32_t mn2 = E::kInfPattern * 0x10001u, mx2 = 0u;
        uint4* xp = xpark + (n_a % 3u) * (p.park_stride / 16u);
        cp_async_wait_all();  // this thread's own copies: nobody else touches these 64 bytes
        uint32_t x[16];
#pragma unroll
        for (uint32_t j = 0; j < 4; ++j) {
          const uint4 c = j < nvalid ? xp[park_index(nt, u, j)] : make_uint4(0u, 0u, 0u, 0u);
          x[4 * j + 0] = c.x;
          x[4 * j + 1] = c.y;
          x[4 * j + 2] = c.z;
          x[4 * j + 3] = c.w;
        }
        bitmap_cur = split_group<BF16>(x, nvalid, p.thr16 * 0x10001u, mn2, mx2);
        cnt_cur = __popc(bitmap_cur);
        if (SV) {
          // min / max of the signed values of T_below instead (outlier slots are +0 by now): as order keys
          mn2 = 0xffffffffu;
          mx2 = 0u;
#pragma unroll
          for (uint32_t i = 0; i < 16; ++i) {
            if (FULL || (i >> 2) < nvalid) {
              const uint32_t key2 = order_keys2(x[i]);
              mn2 = __vminu2(mn2, key2);
              mx2 = __vmaxu2(mx2, key2);
            }
          }
        }
        if (bitmap_cur != 0u) {
          // the original pattern of the group's first outlier, from the parked row while it still holds it:
          // the CSR entry is written an iteration later, and most groups with an outlier have just one
          const uint32_t b = static_cast<uint32_t>(__ffs(bitmap_cur) - 1);
          first_cur = reinterpret_cast<const uint16_t*>(xp)[8u * park_index(nt, u, b >> 3) + (b & 7u)];
        }
        if (bitmap_cur != 0u || nvalid < 4u) {  // outlier slots become +0 (and the chunks past the end of the row)
#pragma unroll
          for (uint32_t j = 0; j < 4; ++j) xp[park_index(nt, u, j)] = make_uint4(x[4 * j], x[4 * j + 1], x[4 * j + 2], x[4 * j + 3]);
        }
        const uint32_t mnv = __reduce_min_sync(kFull, min(mn2 & 0xffffu, mn2 >> 16));
        const uint32_t mxv = __reduce_max_sync(kFull, max(mx2 & 0xffffu, mx2 >> 16));
        const uint32_t wcnt = __reduce_add_sync(kFull, cnt_cur);
        if (lane == 0) {
          m.part.warp_min[warp] = mnv;
          m.part.warp_max[warp] = mxv;
          m.part.warp_cnt[warp] = wcnt;
        }
      }
      if (tid == 0) {
        if (have_cur) {
          sh.meta[n_a % kMetaRing].tile = tile_cur;
          sh.next_tile[(n_a + 1u) & 1u] = ticket_ahead;
        }
        if (have_prev) {
          // pass B of row n_a - 1 needs its levels
          wait_beyond(&sh.lv_ready, n_a - 1u, sh, false, 100u);
        }
        // The levels and placement warps may raise abort at any moment.  Thread 0 alone samples it, before the
        // barrier, into a word that nobody else writes: every compute thread then takes the same branch.
        sh.stop[it & 1u] = sh.abort;
        if (heavy_filled != heavy_done) sh.heavy_seen[it & 1u] = sh.heavy_posted;
      }
      compute_barrier(nt);
      if (sh.stop[it & 1u] != 0u) break;
      if (tid == 0) {
        __threadfence_block();
        if (have_cur) sh.a_ready = n_a + 1u;
        sh.packed = n_a - (have_prev ? 1u : 0u);
        if (have_cur && ticket_ahead < p.tokens) ticket_ahead = atomicAdd(&p.ws->ticket, 1u);  // for the row after the next
      }
      const uint32_t tile_next = have_cur ? sh.next_tile[(n_a + 1u) & 1u] : 0xffffffffu;
      if (tile_next < p.tokens) fetch_group(p, xpark, tile_next, (n_a + 1u) % 3u, u, FULL ? 4u : group_chunks(p, u));  // in flight during passes B and C below

      if (have_prev) {
        const uint32_t n = n_a - 1u;
        RowMeta& m = sh.meta[n % kMetaRing];
        const bool divide = m.divide != 0u;
        const int bmax = p.bits[p.n_bits - 1];
        const uint32_t tile_prev = m.tile;
        const uint4* xp = xpark + (n % 3u) * (p.park_stride / 16u);
        uint32_t r[8];
        int best_ci = p.n_bits - 1;  // the chosen candidate: its level is read again where it is needed
        int bstar = bmax;
        const Level top = m.lv[p.n_bits - 1];
        if (divide) {
          // ---- a row whose scale or zero-point is outside the range of the FMA quotient and of the packed
          //      integer steps (rare): Algorithm 1 with the division instruction, in loops that are not unrolled ----
          const uint32_t* xw = reinterpret_cast<const uint32_t*>(xp);
          for (int ci = p.n_bits - 2; ci >= 0; --ci) {
            const Level low = m.lv[ci];
            uint32_t S = rolled_distortion<BF16, SV>(xw, nt, u, top, low, bmax - p.bits[ci], 4u * (FULL ? 4u : group_chunks(p, u)));
            S = __reduce_add_sync(kFull, S);
            if (lane == 0 && S != 0u) atomicAdd(&m.S[ci], static_cast<int>(S));
            compute_barrier(nt);
            if (m.S[ci] > p.s_max) break;  // keep the last level that passed
            bstar = p.bits[ci];
            best_ci = ci;
          }
          const Planes8 pl = rolled_pack<BF16, SV>(xw, nt, u, m.lv[best_ci], 4u * (FULL ? 4u : group_chunks(p, u)));
#pragma unroll
          for (int k = 0; k < 8; ++k) r[k] = pl.v[k];
        } else {
          // ---- Algorithm 1, one candidate per turn.  The first turn also leaves the top-level bytes (what pass C
          //      packs when the first lower candidate fails, the usual case, and where later turns take the
          //      top-level codes from); every turn leaves its candidate's codes, which become the planes when
          //      that candidate is the last to pass.  With one candidate only, the turn runs for its bytes alone. ----
          uint32_t tb[8], lb[8];
          int ci = p.n_bits - 2;
          {
            uint32_t y[16];
#pragma unroll
            for (uint32_t j = 0; j < 4; ++j) {
              const uint4 c = xp[park_index(nt, u, j)];
              y[4 * j + 0] = c.x;
              y[4 * j + 1] = c.y;
              y[4 * j + 2] = c.z;
              y[4 * j + 3] = c.w;
            }
            const int c0 = ci >= 0 ? ci : 0;
            const Level low = m.lv[c0];
            uint32_t S = distortion_first<BF16, SV>(y, make_level2(top), make_level2(low), bmax - p.bits[c0], tb, lb,
                                                    (FULL || !SV) ? 4u : group_chunks(p, u));
            if (ci >= 0) {
              S = __reduce_add_sync(kFull, S);
              if (lane == 0 && S != 0u) atomicAdd(&m.S[ci], static_cast<int>(S));
            }
          }
          // pass C at the top level right away: the usual outcome, and work to do while the other warps
          // arrive at the barrier (a row that goes lower transposes once more, below)
          planes_of_bytes(tb, r);
          bool passed = false;
          if (ci >= 0) {
            compute_barrier(nt);
            passed = m.S[ci] <= p.s_max;
          }
          if (passed) {
            bstar = p.bits[ci];
            best_ci = ci;
            for (--ci; ci >= 0; --ci) {
              uint32_t y[16], ql[8];
#pragma unroll
              for (uint32_t j = 0; j < 4; ++j) {
                const uint4 c = xp[park_index(nt, u, j)];
                y[4 * j + 0] = c.x;
                y[4 * j + 1] = c.y;
                y[4 * j + 2] = c.z;
                y[4 * j + 3] = c.w;
              }
              const Level low = m.lv[ci];
              uint32_t S = distortion_next<BF16, SV>(y, tb, make_level2(low), bmax - p.bits[ci], ql,
                                                     (FULL || !SV) ? 4u : group_chunks(p, u));
              S = __reduce_add_sync(kFull, S);
              if (lane == 0 && S != 0u) atomicAdd(&m.S[ci], static_cast<int>(S));
              compute_barrier(nt);
              if (m.S[ci] > p.s_max) break;  // keep the last level that passed
              bstar = p.bits[ci];
              best_ci = ci;
#pragma unroll
              for (int k = 0; k < 8; ++k) lb[k] = ql[k];
            }
            // the chosen candidate's codes with the signs of the top-level bytes
#pragma unroll
            for (int k = 0; k < 8; ++k) tb[k] = SV ? lb[k] : (lb[k] | (tb[k] & 0x80808080u));
            planes_of_bytes(tb, r);
          }
        }
        const uint32_t row_cnt = m.row_cnt;
        const uint32_t agg_w = static_cast<uint32_t>(bstar) * p.lay.wpp;
        // more outliers than the slot's list holds: into a side buffer when one is free
        const bool to_heavy = row_cnt > p.csr_cap && heavy_filled == heavy_done;
        if (tid == 0) {
          // the row's sizes are known: let the rows behind it see them
          publish_aggregate(p, gen4, tile_prev, agg_w, row_cnt);
          m.heavy = to_heavy ? 1u : 0u;
          m.bstar = static_cast<uint32_t>(bstar);
          m.agg_w = agg_w;
          m.scale = m.lv[best_ci].s;
          m.zp = m.lv[best_ci].zp;
        }
        // ---- the slot that the row's planes and CSR entries go to must have been emptied by the placement of
        //      row n - p.ring.  Every thread looks for itself, and only now: the row's sizes are published
        //      already, so a CTA whose ring is full does not keep the rows behind it (in other CTAs) waiting
        //      for this row's sizes on top of its own wait. ----
        const bool slot_free = n < p.ring || wait_beyond(&sh.placed, n - p.ring, sh, false, 100u);
        // ---- planes of the chosen level into the row's slot, in blob order ----
        if (slot_free && (FULL || u < p.units)) store_planes<SV>(planes + slot * (p.planes_stride / 4u) + u * static_cast<uint32_t>(bstar), r, bstar, true);
        // ---- a row with more outliers than the list holds leaves its groups' bitmaps in a side buffer, or, when
        //      both are taken, in the list itself (it has room for at least two words per compute thread), where
        //      the placement warp makes the entries from them ----
        if (to_heavy) {
          sh.heavy_bm[u] = bitmap_prev;
          if (lane == 0) sh.heavy_wcnt[warp] = m.part.warp_cnt[warp];
          if (tid == 0) sh.heavy_tile = tile_prev;
          ++heavy_filled;
        } else if (slot_free && row_cnt > p.csr_cap) {
          csr[slot * p.csr_cap + u] = bitmap_prev;
        }
        // ---- CSR entries of T_above into the row's list: ascending columns, original patterns ----
        const uint32_t flagged = __ballot_sync(kFull, cnt_prev != 0u);
        if (flagged != 0u) {
          uint32_t before;  // outliers in the lanes below this one
          if (__ballot_sync(kFull, cnt_prev > 1u) == 0u) {
            before = __popc(flagged & ((1u << lane) - 1u));  // one per flagged lane: its rank among them
          } else {
            uint32_t incl = cnt_prev;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
              const uint32_t v = __shfl_up_sync(kFull, incl, d);
              if (lane >= static_cast<uint32_t>(d)) incl += v;
            }
            before = incl - cnt_prev;
          }
          if (slot_free && cnt_prev != 0u && row_cnt <= p.csr_cap) {
            uint32_t* list = csr + slot * p.csr_cap;
            const uint16_t* x16 = p.x + static_cast<size_t>(tile_prev) * p.hidden;
            uint32_t at = m.part.warp_cnt[warp] + before;
            uint32_t bm = bitmap_prev;
            list[at++] = ((32u * u + static_cast<uint32_t>(__ffs(bm) - 1)) << 16) | first_prev;
            bm &= bm - 1u;
            if (__popc(bm) <= 5) {
              while (bm != 0u) {  // further outliers of the group: read from the input again
                const uint32_t e = 32u * u + static_cast<uint32_t>(__ffs(bm) - 1);
                bm &= bm - 1u;
                list[at++] = (e << 16) | x16[e];
              }
            } else {
              // many: the group's 64 bytes in one round trip instead of one dependent load per outlier
              const uint4* g = reinterpret_cast<const uint4*>(x16) + 4u * u;
              const uint32_t nv = FULL ? 4u : group_chunks(p, u);
              uint4 v[4];
#pragma unroll
              for (uint32_t j = 0; j < 4; ++j) v[j] = j < nv ? g[j] : make_uint4(0u, 0u, 0u, 0u);
              for_each_flagged(bm, v, 32u * u, [&](uint32_t entry) { list[at++] = entry; });
            }
          }
        }
        fence_proxy_async_smem();  // the planes are about to be read by the bulk-copy engine
        slot = slot + 1u == p.ring ? 0u : slot + 1u;
      }
      // the row in the side buffer, once the placement warp has posted its offset (as thread 0 saw it before this
      // iteration's barrier).  Here, after pass C, so that the buffer is not refilled in the iteration that empties it:
      // the next pass C comes after the next barrier.
      if (heavy_filled != heavy_done && sh.heavy_seen[it & 1u] > heavy_done) {
        emit_heavy();
        ++heavy_done;
      }
      have_prev = have_cur;
      bitmap_prev = bitmap_cur;
      cnt_prev = cnt_cur;
      first_prev = first_cur;
      if (have_cur) ++n_a;
      tile_cur = tile_next;
    }
    compute_barrier(nt);
    if (tid == 0) {
      __threadfence_block();
      sh.packed = n_a - (have_prev ? 1u : 0u);  // have_prev is still set only when the loop was left by an abort
      __threadfence_block();
      sh.finished = 1u;
    }
    // rows still in the side buffers: wait for the placement warp to post their offsets
    while (heavy_done < heavy_filled) {
      if (tid == 0) sh.heavy_seen[0] = wait_beyond(&sh.heavy_posted, heavy_done, sh, false, 200u) ? 1u : 0u;
      compute_barrier(nt);
      const bool posted = sh.heavy_seen[0] != 0u;
      if (posted) emit_heavy();
      ++heavy_done;
      compute_barrier(nt);  // before thread 0 writes heavy_seen[0] again
      if (!posted) break;   // the CTA aborted
    }
  } else if (warp == nwarps) {
    // ================================ levels warp ================================
    for (uint32_t n = 0;; ++n) {
      if (!wait_beyond(&sh.a_ready, n, sh, true, 500u)) break;
      __threadfence_block();
      RowMeta& m = sh.meta[n % kMetaRing];
      const uint32_t divide = row_levels<BF16, (kPipeMaxThreads - 64) / 32, SV>(p, m.part, nwarps, lane, m.lv, m.S, &m.row_cnt);
      if (lane == 0) m.divide = divide;
      __syncwarp();
      if (lane == 0) {
        __threadfence_block();
        sh.lv_ready = n + 1u;
      }
    }
  } else {
    // ================================ placement warp ================================
    uint32_t slot = 0u;  // n mod p.ring
    for (uint32_t n = 0;; ++n, slot = slot + 1u == p.ring ? 0u : slot + 1u) {
      if (!wait_beyond(&sh.packed, n, sh, true, 1500u)) break;
      __threadfence_block();
      const RowMeta& m = sh.meta[n % kMetaRing];
      const uint32_t tile = m.tile, agg_w = m.agg_w, row_cnt = m.row_cnt;
      // Everything the stores below need from shared memory is read before the look-back, whose round trips it then
      // overlaps with: the token's fields (one per lane: a lone warp pays for every divergent branch, so each lane
      // selects its field's address and value and one store serves them all) and, for the usual row, whose CSR
      // entries number 64 at most, the entries themselves, two per lane.
      const uint32_t heavy = m.heavy;
      const bool short_list = heavy == 0u && row_cnt <= 64u && row_cnt <= p.csr_cap;
      uint32_t e0 = 0u, e1 = 0u;
      if (short_list) {
        const uint32_t* list = csr + slot * p.csr_cap;
        if (lane < row_cnt) e0 = list[lane];
        if (lane + 32u < row_cnt) e1 = list[lane + 32u];
      }
      // lanes 1 .. 4: scale, zero-point, word_off[tile + 1], out_ptr[tile + 1]; lanes 5, 6 (first token only): the two leading zeros
      unsigned long long field_off = 0ull;
      uint32_t field_val = 0u;
      bool field = false;
      if (lane == 1u) { field_off = p.lay.off_scale + 4ull * tile; field_val = __float_as_uint(m.scale); field = true; }
      if (lane == 2u) { field_off = p.lay.off_zp + 4ull * tile; field_val = static_cast<uint32_t>(m.zp); field = true; }
      if (lane == 3u) { field_off = p.lay.off_word_off + 4ull * (tile + 1u); field_val = agg_w; field = true; }
      if (lane == 4u) { field_off = p.lay.off_out_ptr + 4ull * (tile + 1u); field_val = row_cnt; field = true; }
      if (lane == 5u && tile == 0u) { field_off = p.lay.off_word_off; field = true; }
      if (lane == 6u && tile == 0u) { field_off = p.lay.off_out_ptr; field = true; }
      const uint32_t bstar8 = m.bstar;
      uint32_t word_off = 0, out_base = 0;
      const int st = resolve_prefix<1>(p, gen4, tile, agg_w, row_cnt, lane, &word_off, &out_base, lookback_limit(p));
      if (st != TSQ_OK) {
        if (lane == 0) {
          publish(p, gen4 | kFlagAbort, tile, 0u, 0u);
          if (st > 0) atomicCAS(&p.ws->err, 0u, static_cast<uint32_t>(st));
        }
      } else {
        uint32_t* wdst = reinterpret_cast<uint32_t*>(p.blob + p.lay.off_words) + word_off;
        const uint32_t* src = planes + slot * (p.planes_stride / 4u);
        if (p.vec_store != 0u) {
          if (lane == 0) {
            bulk_s2g(wdst, src, agg_w * 4u);
            bulk_commit();
          }
        } else {  // runs of words that are not multiples of 16 bytes: plain stores
          for (uint32_t w = lane; w < agg_w; w += 32) wdst[w] = src[w];
        }
        // the token's fields
        if (lane == 3u) field_val += word_off;
        if (lane == 4u) field_val += out_base;
        if (field) *reinterpret_cast<uint32_t*>(p.blob + field_off) = field_val;
        if (lane == 0) reinterpret_cast<uint8_t*>(p.blob + p.lay.off_bits)[tile] = static_cast<uint8_t>(bstar8);
        if (row_cnt != 0u) {
          uint32_t* o_outl = reinterpret_cast<uint32_t*>(p.blob + p.lay.off_outl);
          bool overflow = false;
          if (short_list) {
            const unsigned long long at0 = static_cast<unsigned long long>(out_base) + lane, at1 = at0 + 32ull;
            if (lane < row_cnt) {
              if (at0 < p.lay.outlier_capacity) {
                o_outl[at0] = e0;
              } else {
                overflow = true;
              }
            }
            if (lane + 32u < row_cnt) {
              if (at1 < p.lay.outlier_capacity) {
                o_outl[at1] = e1;
              } else {
                overflow = true;
              }
            }
          } else if (heavy != 0u) {
            // the compute threads write this row's entries: tell them where
            if (lane == 0) {
              sh.heavy_base = out_base;
              __threadfence_block();
              sh.heavy_posted = sh.heavy_posted + 1u;
            }
          } else if (row_cnt <= p.csr_cap) {
            const uint32_t* list = csr + slot * p.csr_cap;
            for (uint32_t i = lane; i < row_cnt; i += 32) {
              const unsigned long long at = static_cast<unsigned long long>(out_base) + i;
              if (at < p.lay.outlier_capacity) {
                o_outl[at] = list[i];
              } else {
                overflow = true;
              }
            }
          } else {
            // more outliers than the list holds: the list holds the groups' bitmaps instead.  32 groups per turn:
            // a scan of the counts, then every lane reads its group's 64 bytes from the input again (one round
            // trip for the whole turn) and writes its entries
            const uint32_t* bms = csr + slot * p.csr_cap;
            const uint4* xrow4 = reinterpret_cast<const uint4*>(p.x + static_cast<size_t>(tile) * p.hidden);
            unsigned long long pos = out_base;
            for (uint32_t g0 = 0; g0 < nt; g0 += 32u) {
              const uint32_t g = g0 + lane;
              const uint32_t bm = bms[g];
              const uint32_t cnt = __popc(bm);
              uint32_t incl = cnt;
#pragma unroll
              for (int d = 1; d < 32; d <<= 1) {
                const uint32_t up = __shfl_up_sync(kFull, incl, d);
                if (lane >= static_cast<uint32_t>(d)) incl += up;
              }
              unsigned long long at = pos + (incl - cnt);
              pos += __shfl_sync(kFull, incl, 31);
              if (bm != 0u) {
                uint4 v[4];
#pragma unroll
                for (uint32_t j = 0; j < 4; ++j) v[j] = 4u * g + j < p.chunks ? xrow4[4u * g + j] : make_uint4(0u, 0u, 0u, 0u);
                for_each_flagged(bm, v, 32u * g, [&](uint32_t entry) {
                  if (at < p.lay.outlier_capacity) {
                    o_outl[at] = entry;
                  } else {
                    overflow = true;
                  }
                  ++at;
                });
              }
            }
          }
          if (__any_sync(kFull, overflow) && lane == 0) {
            atomicCAS(&p.ws->err, 0u, static_cast<uint32_t>(TSQ_ERR_OUTLIER_OVERFLOW));
          }
        }
      }
      __syncwarp();
      if (lane == 0) {
        // A slot may be refilled once the bulk store has read it.  The wait is for the store of the row
        // before this one, which has had a whole row's time to finish: this row's store is left in flight
        // and its slot is given back one row later (plain stores have read their slot already).
        if (p.vec_store != 0u) bulk_wait_read_but_one();
        __threadfence_block();
        sh.placed = p.vec_store != 0u ? n : n + 1u;
      }
    }
    if (lane == 0) bulk_wait_all();  // shared memory must outlive the stores that read it
  }

  __syncthreads();
  if (tid == 0) {
    if (sh.abort != 0u) atomicCAS(&p.ws->err, 0u, static_cast<uint32_t>(TSQ_ERR_TIMEOUT));
    finish_call(p, gen4);
  }
}

}  // namespace

// The pipelined kernel is built for CTAs of up to kPipeMaxThreads threads (rows of up to 8192 elements)
// and may use up to 102 registers per thread; longer rows take encode_rows_kernel.
template <bool SV>
static const void* pipe_kernel_of(bool bf16, bool full) {
  if (full) {
    return bf16 ? reinterpret_cast<const void*>(&encode_pipe_kernel<true, true, kPipeMaxThreads, 2, SV>)
                : reinterpret_cast<const void*>(&encode_pipe_kernel<false, true, kPipeMaxThreads, 2, SV>);
  }
  return bf16 ? reinterpret_cast<const void*>(&encode_pipe_kernel<true, false, kPipeMaxThreads, 2, SV>)
              : reinterpret_cast<const void*>(&encode_pipe_kernel<false, false, kPipeMaxThreads, 2, SV>);
}
static const void* pipe_kernel(bool bf16, bool full, bool sv) { return sv ? pipe_kernel_of<true>(bf16, full) : pipe_kernel_of<false>(bf16, full); }

cudaError_t encode_pipe_attrs(bool bf16, bool full, bool sv, int threads, size_t smem, int* blocks_per_sm) {
  if (threads > kPipeMaxThreads) return cudaErrorInvalidValue;
  const void* fn = pipe_kernel(bf16, full, sv);
  // the attribute belongs to the kernel on the current device, not to a plan: it only ever grows, so
  // that every plan can launch
  static std::mutex mu;
  static size_t granted[kMaxDevices][2][2][2] = {};
  {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(mu);
    size_t& have = granted[dev][bf16 ? 1 : 0][full ? 1 : 0][sv ? 1 : 0];
    if (smem > have) {
      e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
      if (e != cudaSuccess) return e;
      have = smem;
    }
  }
  return cudaOccupancyMaxActiveBlocksPerMultiprocessor(blocks_per_sm, fn, threads, smem);
}

template <bool SV>
static void launch_pipe_variant(const EncodeParams& p, bool full, int grid, int threads, size_t smem, cudaStream_t stream) {
  const bool bf16 = p.dtype == TSQ_BF16;
  if (full) {
    if (bf16) {
      encode_pipe_kernel<true, true, kPipeMaxThreads, 2, SV><<<grid, threads, smem, stream>>>(p);
    } else {
      encode_pipe_kernel<false, true, kPipeMaxThreads, 2, SV><<<grid, threads, smem, stream>>>(p);
    }
  } else if (bf16) {
    encode_pipe_kernel<true, false, kPipeMaxThreads, 2, SV><<<grid, threads, smem, stream>>>(p);
  } else {
    encode_pipe_kernel<false, false, kPipeMaxThreads, 2, SV><<<grid, threads, smem, stream>>>(p);
  }
}

cudaError_t launch_encode_pipe(const EncodeParams& p, bool full, int grid, int threads, size_t smem, cudaStream_t stream) {
  if (threads > kPipeMaxThreads) return cudaErrorInvalidValue;
  if (p.variant != 0u) {
    launch_pipe_variant<true>(p, full, grid, threads, smem, stream);
  } else {
    launch_pipe_variant<false>(p, full, grid, threads, smem, stream);
  }
  return cudaGetLastError();
}

template <bool SV>
static void launch_rows_variant(const EncodeParams& p, int grid, int threads, int upt, cudaStream_t stream) {
  const bool bf16 = p.dtype == TSQ_BF16;
  if (upt == 1 && threads <= 256) {
    if (bf16) {
      encode_rows_kernel<true, 1, 256, SV><<<grid, threads, 0, stream>>>(p);
    } else {
      encode_rows_kernel<false, 1, 256, SV><<<grid, threads, 0, stream>>>(p);
    }
  } else if (upt == 1) {
    if (bf16) {
      encode_rows_kernel<true, 1, 1024, SV><<<grid, threads, 0, stream>>>(p);
    } else {
      encode_rows_kernel<false, 1, 1024, SV><<<grid, threads, 0, stream>>>(p);
    }
  } else {
    if (bf16) {
      encode_rows_kernel<true, 2, 1024, SV><<<grid, threads, 0, stream>>>(p);
    } else {
      encode_rows_kernel<false, 2, 1024, SV><<<grid, threads, 0, stream>>>(p);
    }
  }
}

cudaError_t launch_encode_rows(const EncodeParams& p, int grid, int threads, int upt, cudaStream_t stream) {
  if (p.variant != 0u) {
    launch_rows_variant<true>(p, grid, threads, upt, stream);
  } else {
    launch_rows_variant<false>(p, grid, threads, upt, stream);
  }
  return cudaGetLastError();
}

}  // namespace tsq
