// tsq encode kernel: threshold splitting (Eq. "ts") + token-wise TAB-Q (Algorithm 1 on AIQ,
// Eq. "Proposed") + bit-plane packing + CSR emission, fused into one persistent kernel.
//
// One WARP works on one token row at a time, and no two warps ever synchronise with each other:
// a warp takes the next row by an atomic ticket, fetches it into its own shared-memory slot with
// one bulk asynchronous copy (completion on the warp's own mbarrier), runs every pass of the
// method on that copy, and sends the row's planes to the blob with one bulk asynchronous store.
// The input is therefore read from HBM exactly once, and while one warp waits (for its copy, or
// for the placement of its output) the other warps of the SM keep the issue slots busy.
//
// Passes over the slot:
//   A      threshold split: per-token min / max of the inlier magnitudes; every outlier is copied
//          (column, original pattern) to the warp's stash in column order and its slot is set to +0,
//          which is what T_below holds there, so the later passes need no mask;
//   B      Algorithm 1: AIQ codes at the top level and at each lower candidate, distortion sums;
//   C      codes at the chosen level -> bytes (code << 1 | sign) -> 8 x 32 bit transpose -> the
//          group's b* plane words, written over the front of the slot itself (group g's words end
//          before group g's input begins, and a warp reads 32 groups before it writes them);
//   then the placement is looked up and slot and stash leave for the blob.
//
// Variable-length placement: where a token's planes and CSR entries start is an exclusive prefix
// sum over all earlier tokens.  It is resolved with a decoupled look-back over per-token
// descriptors in the workspace.  Tickets are handed out in row order, so a row only ever waits
// for rows held by warps that are already running.  A row publishes its own sizes right after
// pass B and looks back only after pass C, so that the wait for slower predecessors overlaps its
// own packing.  A look-back step reads 256 descriptors at once (eight independent loads per
// lane): with well over a hundred rows finishing per microsecond, a narrower window cannot reach
// the nearest published prefix within one memory round trip.  Every wait is bounded and fails
// into a status word.
//
// Arithmetic contract: the codes equal  clamp(rint(m / s) - zp, 0, Qmax)  with the IEEE binary32
// quotient m / s.  Three evaluations of it exist, chosen per row:
//   kFast     rint(m * r) with r = fl(1/s), one FMA against 1.5 * 2^23.  It can differ from the
//             contract only when m / s lies within a relative 2^-22 of a rounding boundary k + 1/2
//             (exact ties included: 16-bit inputs make m / s land exactly on k + 1/2 quite often).
//             16-bit values are at least 2^-11 apart, so for each boundary only its two
//             neighbouring 16-bit values can be affected; those are examined per row, a cheap
//             distance test first and the true division for the few that fail it.
//   kRefined  for a row where any of them really disagrees: the correctly rounded quotient from
//             q0 = fl(m * r), the exact residual m - q0 * s (one FMA) and q = fl(q0 + residual * r)
//             (the classical FMA division step, exact when r is the correctly rounded reciprocal
//             and nothing over- or underflows), then the same 1.5 * 2^23 rounding.
//   kDivide   the division instruction itself, for rows whose scale is so large or so small that
//             the intermediate products of the other two could leave the normal range, or whose
//             zero-point does not fit the packed 16-bit integer steps of the other two.

#include "tsq_device.cuh"
#include "tsq_internal.h"

namespace tsq {
namespace {

constexpr float kRoundMagic = 8388608.0f;  // 2^23: adding it to 0 <= y < 2^23 rounds y to an integer, ties to even
constexpr uint32_t kRoundMagicHi = 0x4B00u;  // upper 16 bits of the pattern of 2^23
constexpr uint32_t kLookbackPollLimit = 1u << 20;
constexpr uint32_t kCopyPollLimit = 1u << 20;
constexpr int kLookbackDepth = 8;  // descriptors each lane reads per look-back step

// AIQ parameters of one candidate level for one row (Eq. "Proposed").
struct Level {
  float s;       // scale
  float r;       // fl(1 / s)
  int zp;        // zero-point rint(m_min / s)
  int qmax;      // 2^(b-1) - 1
  uint32_t nz2;  // -zp in the low half, -zp - kRoundMagicHi in the high half (see codes2)
  uint32_t qm2;  // qmax in both 16-bit halves
  bool fast;     // scale and zero-point in the range where the FMA paths are provably safe
};

enum Mode : int { kFast = 0, kRefined = 1, kDivide = 2 };

__device__ __forceinline__ Level make_level(float mmin, float mmax, int b) {
  Level c;
  c.qmax = (1 << (b - 1)) - 1;
  const float range = __fsub_rn(mmax, mmin);
  c.s = range > 0.0f ? __fdiv_rn(range, static_cast<float>(c.qmax)) : (mmax > 0.0f ? mmax : 1.0f);
  c.zp = __float2int_rn(__fdiv_rn(mmin, c.s));
  c.r = __fdiv_rn(1.0f, c.s);
  c.nz2 = (static_cast<uint32_t>(-c.zp) & 0xffffu) | (static_cast<uint32_t>(-c.zp - static_cast<int>(kRoundMagicHi)) << 16);
  c.qm2 = static_cast<uint32_t>(c.qmax) * 0x10001u;
  // rint(m / s) <= zp + qmax + 1 must stay a small positive 16-bit integer for the packed steps
  c.fast = (c.s >= 0x1p-60f) && (c.s <= 0x1p60f) && (c.zp < 12000);
  return c;
}

// Code of one magnitude (scalar form: boundary checks only).
template <int MODE>
__device__ __forceinline__ int code_of(float m, const Level& c) {
  int k;
  if (MODE == kFast) {
    k = (__float_as_int(fmaf(m, c.r, kRoundMagic)) & 0xffff) - c.zp;
  } else {
    k = __float2int_rn(__fdiv_rn(m, c.s)) - c.zp;
  }
  return __vimin_s32_relu(k, c.qmax);  // clamp to [0, qmax]
}

// Codes of the two elements of a 16-bit pair (sign bits ignored), as two 16-bit integers.
template <bool BF16, int MODE>
__device__ __forceinline__ uint32_t codes2(uint32_t x, const Level& c) {
  using E = Elem<BF16>;
  const float lo = fabsf(E::lo_f32(x)), hi = fabsf(E::hi_f32(x));
  if (MODE == kDivide) {
    const int klo = __vimin_s32_relu(__float2int_rn(__fdiv_rn(lo, c.s)) - c.zp, c.qmax);
    const int khi = __vimin_s32_relu(__float2int_rn(__fdiv_rn(hi, c.s)) - c.zp, c.qmax);
    return static_cast<uint32_t>(klo) | (static_cast<uint32_t>(khi) << 16);
  }
  float tlo, thi;
  if (MODE == kFast) {
    tlo = fmaf(lo, c.r, kRoundMagic);
    thi = fmaf(hi, c.r, kRoundMagic);
  } else {
    const float q0 = __fmul_rn(lo, c.r), q1 = __fmul_rn(hi, c.r);
    tlo = __fadd_rn(fmaf(fmaf(-q0, c.s, lo), c.r, q0), kRoundMagic);  // fl(lo / s), then to an integer
    thi = __fadd_rn(fmaf(fmaf(-q1, c.s, hi), c.r, q1), kRoundMagic);
  }
  // pattern of 2^23 + k = 0x4B000000 + k.  thi * 2^16 + tlo (mod 2^32) = (0x4B00 + k_lo's carry-free
  // neighbour k_hi) << 16 | k_lo; the constant in the high half is taken off together with zp.
  const uint32_t k2 = __float_as_uint(thi) * 65536u + __float_as_uint(tlo);
  return __viaddmin_s16x2_relu(k2, c.nz2, c.qm2);  // clamp(k - zp, 0, qmax) in both halves
}

// Does the fast path disagree with the true division for a 16-bit value next to rounding
// boundary (zp + j - 1/2) * s ?  Only values inside [pmin, pmax] can occur in the row.
template <bool BF16>
__device__ __forceinline__ bool boundary_disagrees(const Level& c, int j, uint32_t pmin, uint32_t pmax) {
  using E = Elem<BF16>;
  const float h = static_cast<float>(c.zp + j) - 0.5f;
  if (!(h > 0.0f)) return false;
  const float centre = __fmul_rn(h, c.s);
  const uint32_t plo = E::pattern_rd(centre);
  const float margin = __fmul_rn(h, 0x1p-21f);
  bool bad = false;
#pragma unroll
  for (uint32_t d = 0; d < 2; ++d) {
    const uint32_t pat = plo + d;
    if (pat >= pmin && pat <= pmax) {
      const float m = E::pattern_f32(pat);
      // |m * r - h| > h * 2^-21 puts m / s more than h * 2^-22 away from the boundary: both paths agree
      if (fabsf(__fsub_rn(__fmul_rn(m, c.r), h)) <= margin) bad |= code_of<kFast>(m, c) != code_of<kDivide>(m, c);
    }
  }
  return bad;
}

// Examine the boundaries of one or two levels, spread over the lanes of the warp.
template <bool BF16>
__device__ __forceinline__ bool levels_disagree(const Level* first, const Level& second, uint32_t pmin, uint32_t pmax,
                                                uint32_t lane) {
  const int n_first = first ? first->qmax + 2 : 0;
  const int n_items = n_first + second.qmax + 2;
  bool bad = false;
  for (int w = static_cast<int>(lane); w < n_items; w += 32) {
    bad |= (w < n_first) ? boundary_disagrees<BF16>(*first, w, pmin, pmax)
                         : boundary_disagrees<BF16>(second, w - n_first, pmin, pmax);
  }
  return __any_sync(kFull, bad);
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

// Pass B. Numerator of Algorithm 1's distortion for one row: sum |(q0 >> sh) - q|, whole warp.
// The terms are non-negative, so the pass stops as soon as the running sum exceeds s_max: the
// returned value is then only known to be > s_max, which is all the caller asks.
template <bool BF16, int MODE>
__device__ __forceinline__ int distortion(const uint4* row, const EncodeParams& p, const Level& top, const Level& low,
                                          int sh, uint32_t lane) {
  const uint32_t shmask = (0xffffu >> sh) * 0x10001u;
  uint32_t S = 0;
  int total = 0;
  for (uint32_t base = 0; base < p.units; base += 32) {
    const uint32_t u = base + lane;
    uint32_t S2 = 0;  // two 16-bit partial sums: at most 16 * 127 each per unit
    if (u < p.units) {
#pragma unroll
      for (uint32_t j = 0; j < 4; ++j) {
        const uint32_t cidx = 4u * u + j;
        if (cidx >= p.chunks) continue;
        const uint4 c = row[cidx];
        const uint32_t x[4] = {c.x, c.y, c.z, c.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const uint32_t a = (codes2<BF16, MODE>(x[i], top) >> sh) & shmask;
          const uint32_t q = codes2<BF16, MODE>(x[i], low);
          S2 += max_s16x2(a, q) - min_s16x2(a, q);
        }
      }
    }
    S += (S2 & 0xffffu) + (S2 >> 16);
    total = static_cast<int>(__reduce_add_sync(kFull, S));
    if (total > p.s_max) break;
  }
  return total;
}

// Pass C. Codes of the row at the chosen level as bytes (code | sign << 7), transposed into
// bit-planes and written over the front of the slot: group g's b* words go to words
// g * b* .. g * b* + b* - 1, plane 0 = sign, plane 1 + k = bit k of the code.
template <bool BF16, int MODE>
__device__ __forceinline__ void pack_row(uint4* row, const EncodeParams& p, const Level& lv, int bstar, uint32_t lane) {
  uint32_t* out = reinterpret_cast<uint32_t*>(row);
  for (uint32_t base = 0; base < p.units; base += 32) {
    const uint32_t u = base + lane;
    uint4 c[4];
#pragma unroll
    for (uint32_t j = 0; j < 4; ++j) {
      const uint32_t cidx = 4u * u + j;
      c[j] = (u < p.units && cidx < p.chunks) ? row[cidx] : make_uint4(0u, 0u, 0u, 0u);
    }
    __syncwarp();  // all 32 groups are in registers before any of them is overwritten
    if (u >= p.units) continue;
    // b2[j][i]: bytes of elements 8j + 2i (byte 0) and 8j + 2i + 1 (byte 2)
    uint32_t b2[4][4];
#pragma unroll
    for (uint32_t j = 0; j < 4; ++j) {
      const uint32_t x[4] = {c[j].x, c[j].y, c[j].z, c[j].w};
#pragma unroll
      for (int i = 0; i < 4; ++i) b2[j][i] = codes2<BF16, MODE>(x[i], lv) | ((x[i] >> 8) & 0x00800080u);
    }
    // r[i] byte c = element 8c + i
    uint32_t r[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const uint32_t e = b2[1][i] * 256u + b2[0][i];  // bytes: 8*0+2i, 8*1+2i, 8*0+2i+1, 8*1+2i+1
      const uint32_t f = b2[3][i] * 256u + b2[2][i];  // the same for chunks 2 and 3
      r[2 * i] = __byte_perm(e, f, 0x5410);
      r[2 * i + 1] = __byte_perm(e, f, 0x7632);
    }
    transpose8x32(r);  // r[k] = bit k of every byte: k < 7 code bits, k = 7 signs
    uint32_t* dst = out + static_cast<size_t>(u) * bstar;
    if (bstar == 8) {
      reinterpret_cast<uint4*>(dst)[0] = make_uint4(r[7], r[0], r[1], r[2]);
      reinterpret_cast<uint4*>(dst)[1] = make_uint4(r[3], r[4], r[5], r[6]);
    } else if (bstar == 4) {
      reinterpret_cast<uint4*>(dst)[0] = make_uint4(r[7], r[0], r[1], r[2]);
    } else {
      dst[0] = r[7];
#pragma unroll
      for (int k = 0; k < 7; ++k) {
        if (k < bstar - 1) dst[1 + k] = r[k];
      }
    }
  }
}

__device__ __forceinline__ unsigned long long pack_desc(uint32_t tag, uint32_t value) {
  return (static_cast<unsigned long long>(tag) << 32) | value;
}

// Decoupled look-back over the tile descriptors.
// Descriptor of tile t: (generation * 4 + flag) << 32 | payload.  An AGGREGATE payload carries the
// tile's own sizes, (outliers << 15) | plane words; a PREFIX payload carries the inclusive prefix
// of plane words, and the inclusive prefix of outliers sits in prefix_outl[t], stored before the
// descriptor with a fence between the two.
__device__ __forceinline__ void publish_aggregate(const EncodeParams& p, uint32_t gen4, uint32_t tile, uint32_t agg_w,
                                                  uint32_t agg_o, uint32_t lane) {
  if (tile > 0 && lane == 0) st_relaxed_u64(p.desc + tile, pack_desc(gen4 | kFlagAggregate, (agg_o << 15) | agg_w));
}

// Run by one full warp for its own tile, after publish_aggregate: walk back to the nearest
// published prefix, then publish this tile's own.
// Returns TSQ_OK, TSQ_ERR_TIMEOUT (gave up) or -1 when a predecessor has aborted.
__device__ int resolve_prefix(const EncodeParams& p, uint32_t gen4, uint32_t tile, uint32_t agg_w, uint32_t agg_o,
                              uint32_t lane, uint32_t* excl_w, uint32_t* excl_o) {
  uint32_t base_w = 0, base_o = 0;  // prefix found at the end of the walk
  uint32_t part_w = 0, part_o = 0;  // this lane's share of the aggregates walked over
  if (tile > 0) {
    int pos = static_cast<int>(tile) - 1;  // nearest tile not yet accounted for
    uint32_t polls = 0;
    bool done = false;
    while (!done) {
      unsigned long long v[kLookbackDepth];
#pragma unroll
      for (int k = 0; k < kLookbackDepth; ++k) {
        const int j = pos - (32 * k + static_cast<int>(lane));
        v[k] = j >= 0 ? ld_relaxed_u64(p.desc + j) : pack_desc(gen4 | kFlagPrefix, 0u);  // before tile 0: prefix 0
      }
      int consumed = 32 * kLookbackDepth;
      bool stopped = false;
      int verdict = TSQ_OK;
#pragma unroll
      for (int k = 0; k < kLookbackDepth; ++k) {
        if (stopped) continue;
        const uint32_t tag = static_cast<uint32_t>(v[k] >> 32);
        const uint32_t flag = ((tag & ~3u) == gen4) ? (tag & 3u) : 0u;
        const uint32_t stop = __ballot_sync(kFull, flag != kFlagAggregate);
        const uint32_t first = stop ? static_cast<uint32_t>(__ffs(stop) - 1) : 32u;
        if (lane < first) {
          part_w += static_cast<uint32_t>(v[k]) & 0x7fffu;
          part_o += static_cast<uint32_t>(v[k]) >> 15;
        }
        if (stop == 0u) continue;
        stopped = true;
        const uint32_t first_flag = __shfl_sync(kFull, flag, first);
        if (first_flag == kFlagAbort) {
          verdict = -1;
        } else if (first_flag == kFlagPrefix) {
          base_w = __shfl_sync(kFull, static_cast<uint32_t>(v[k]), first);
          const int j = pos - (32 * k + static_cast<int>(first));
          if (j >= 0) {
            __threadfence();  // pairs with the fence between the two stores of the publisher
            base_o = *reinterpret_cast<volatile const uint32_t*>(p.prefix_outl + j);
          }
          done = true;
        } else {  // not published yet: keep what was walked over, poll again from there
          consumed = 32 * k + static_cast<int>(first);
        }
      }
      if (verdict != TSQ_OK) return verdict;
      if (!done) {
        pos -= consumed;
        if (consumed == 0) {
          // tile `pos` has published nothing yet: watch that one descriptor until it does
          for (;;) {
            uint32_t ready = 0u;
            if (lane == 0) {
              const uint32_t tag = static_cast<uint32_t>(ld_relaxed_u64(p.desc + pos) >> 32);
              ready = ((tag & ~3u) == gen4 && (tag & 3u) != 0u) ? 1u : 0u;
            }
            if (__shfl_sync(kFull, ready, 0) != 0u) break;
            if (++polls > kLookbackPollLimit) return TSQ_ERR_TIMEOUT;
            __nanosleep(polls < 16u ? 250u : 1000u);
          }
        }
      }
    }
    base_w += __reduce_add_sync(kFull, part_w);
    base_o += __reduce_add_sync(kFull, part_o);
  }
  if (lane == 0) {
    p.prefix_outl[tile] = base_o + agg_o;
    __threadfence();
    st_relaxed_u64(p.desc + tile, pack_desc(gen4 | kFlagPrefix, base_w + agg_w));
  }
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
  for (int i = 0; i < 8; ++i) h->bits[i] = (i < p.n_bits) ? static_cast<uint8_t>(p.bits[i]) : 0;
  h->tau = p.tau;
  h->delta = p.delta;
  h->total_words = total_words;
  h->total_outliers = total_outliers;
  h->outlier_capacity = static_cast<uint32_t>(p.lay.outlier_capacity);
}

// All passes of the method on one row held in shared memory.  Returns TSQ_OK, TSQ_ERR_TIMEOUT,
// or 0xffffffff when a predecessor aborted (nothing further to report).  *stored tells the caller
// that a bulk store out of the slot is in flight.
template <bool BF16>
__device__ uint32_t encode_row(const EncodeParams& p, uint32_t gen4, uint32_t tile, uint4* row, uint32_t* stash,
                               uint32_t lane, bool* stored) {
  using E = Elem<BF16>;
  const uint32_t thr2 = p.thr16 * 0x10001u;
  uint16_t* row16 = reinterpret_cast<uint16_t*>(row);

  // ---- pass A: threshold split, min / max of the inlier magnitudes, outliers to the stash ----
  uint32_t mn2 = E::kInfPattern * 0x10001u, mx2 = 0u, row_cnt = 0u;
  for (uint32_t base = 0; base < p.units; base += 32) {
    const uint32_t u = base + lane;
    uint32_t acc[4] = {0u, 0u, 0u, 0u};  // per chunk: bit 2i / bit 17 + 2i flag the low / high element of pair i
    if (u < p.units) {
#pragma unroll
      for (uint32_t j = 0; j < 4; ++j) {
        const uint32_t cidx = 4u * u + j;
        if (cidx >= p.chunks) continue;
        const uint4 c = row[cidx];
        const uint32_t x[4] = {c.x, c.y, c.z, c.w};
        uint32_t m2[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const uint32_t a = x[i] & 0x7fff7fffu;
          const uint32_t mk = E::geu_mask(a, thr2);  // 0xffff in each half with |x| >= tau, NaN included
          m2[i] = a & ~mk;
          acc[j] |= mk & ((1u << (2 * i)) | (1u << (17 + 2 * i)));
        }
        // patterns of non-negative values order like the values: integer min / max
        mx2 = __vimax3_u16x2(mx2, m2[0], m2[1]);
        mx2 = __vimax3_u16x2(mx2, m2[2], m2[3]);
        mn2 = __vimin3_u16x2(mn2, m2[0], m2[1]);
        mn2 = __vimin3_u16x2(mn2, m2[2], m2[3]);
      }
    }
    const uint32_t any = acc[0] | acc[1] | acc[2] | acc[3];
    if (__ballot_sync(kFull, any != 0u) != 0u) {
      uint32_t bitmap = 0u;  // bit e: element 32u + e is an outlier
#pragma unroll
      for (uint32_t j = 0; j < 4; ++j) bitmap |= ((acc[j] | (acc[j] >> 16)) & 0xffu) << (8u * j);
      // where this lane's entries go: exclusive scan of the per-lane counts, columns stay ascending
      const uint32_t cnt = __popc(bitmap);
      uint32_t incl = cnt;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const uint32_t n = __shfl_up_sync(kFull, incl, d);
        if (lane >= static_cast<uint32_t>(d)) incl += n;
      }
      uint32_t at = row_cnt + incl - cnt;
      row_cnt += __shfl_sync(kFull, incl, 31);
      while (bitmap != 0u) {
        const uint32_t e = 32u * u + static_cast<uint32_t>(__ffs(bitmap) - 1);
        bitmap &= bitmap - 1u;
        if (at < p.stash_cap) stash[at] = (e << 16) | row16[e];
        ++at;
        row16[e] = 0;  // T_below holds +0 there
      }
    }
  }
  const uint32_t pmin = __reduce_min_sync(kFull, min(mn2 & 0xffffu, mn2 >> 16));
  const uint32_t pmax = __reduce_max_sync(kFull, max(mx2 & 0xffffu, mx2 >> 16));
  __syncwarp();

  // ---- Algorithm 1: descend the candidate list while the distortion stays within tolerance ----
  const float mmin = E::pattern_f32(pmin), mmax = E::pattern_f32(pmax);
  const int bmax = p.bits[p.n_bits - 1];
  const Level top = make_level(mmin, mmax, bmax);
  Level best = top;
  int bstar = bmax;
  int mode = top.fast ? kFast : kDivide;  // only ever moves towards kDivide within a row
  bool top_checked = false;
  if (p.n_bits == 1 && mode == kFast && levels_disagree<BF16>(nullptr, top, pmin, pmax, lane)) mode = kRefined;
  for (int ci = p.n_bits - 2; ci >= 0; --ci) {
    const int b = p.bits[ci];
    const Level low = make_level(mmin, mmax, b);
    const int sh = bmax - b;
    if (!low.fast) mode = kDivide;
    if (mode == kFast) {
      if (levels_disagree<BF16>(top_checked ? nullptr : &top, low, pmin, pmax, lane)) mode = kRefined;
      top_checked = true;
    }
    const int S = mode == kFast      ? distortion<BF16, kFast>(row, p, top, low, sh, lane)
                  : mode == kRefined ? distortion<BF16, kRefined>(row, p, top, low, sh, lane)
                                     : distortion<BF16, kDivide>(row, p, top, low, sh, lane);
    if (S > p.s_max) break;  // delta > Delta: keep the last level that passed
    bstar = b;
    best = low;
  }

  // ---- this row's sizes are known: let the rows behind it see them, then pack ----
  const uint32_t agg_w = static_cast<uint32_t>(bstar) * p.lay.wpp;
  publish_aggregate(p, gen4, tile, agg_w, row_cnt, lane);
  if (mode == kFast) {
    pack_row<BF16, kFast>(row, p, best, bstar, lane);
  } else if (mode == kRefined) {
    pack_row<BF16, kRefined>(row, p, best, bstar, lane);
  } else {
    pack_row<BF16, kDivide>(row, p, best, bstar, lane);
  }
  fence_proxy_async_smem();  // the packed words are about to be read by the bulk-copy engine
  __syncwarp();

  // ---- placement: exclusive prefix sums over the tokens before this one ----
  uint32_t word_off = 0, out_base = 0;
  const int st = resolve_prefix(p, gen4, tile, agg_w, row_cnt, lane, &word_off, &out_base);
  if (st != TSQ_OK) {
    if (lane == 0) st_relaxed_u64(p.desc + tile, pack_desc(gen4 | kFlagAbort, 0u));
    return st < 0 ? 0xffffffffu : static_cast<uint32_t>(st);
  }
  uint32_t* wdst = reinterpret_cast<uint32_t*>(p.blob + p.lay.off_words) + word_off;
  if (p.bulk_store) {
    if (lane == 0) {
      bulk_s2g(wdst, row, agg_w * 4u);
      bulk_commit();
    }
    *stored = true;
  } else {  // word counts that are not multiples of 16 bytes: plain stores
    const uint32_t* src = reinterpret_cast<const uint32_t*>(row);
    for (uint32_t w = lane; w < agg_w; w += 32) wdst[w] = src[w];
  }
  if (lane == 0) {
    reinterpret_cast<uint8_t*>(p.blob + p.lay.off_bits)[tile] = static_cast<uint8_t>(bstar);
    reinterpret_cast<float*>(p.blob + p.lay.off_scale)[tile] = best.s;
    reinterpret_cast<int32_t*>(p.blob + p.lay.off_zp)[tile] = best.zp;
    uint32_t* o_word_off = reinterpret_cast<uint32_t*>(p.blob + p.lay.off_word_off);
    uint32_t* o_out_ptr = reinterpret_cast<uint32_t*>(p.blob + p.lay.off_out_ptr);
    if (tile == 0) {
      o_word_off[0] = 0;
      o_out_ptr[0] = 0;
    }
    o_word_off[tile + 1] = word_off + agg_w;
    o_out_ptr[tile + 1] = out_base + row_cnt;
  }

  // ---- CSR entries of T_above: ascending columns, original patterns ----
  if (row_cnt != 0u) {
    uint32_t* o_outl = reinterpret_cast<uint32_t*>(p.blob + p.lay.off_outl);
    bool overflow = false;
    if (row_cnt <= p.stash_cap) {
      for (uint32_t i = lane; i < row_cnt; i += 32) {
        const unsigned long long at = static_cast<unsigned long long>(out_base) + i;
        if (at < p.lay.outlier_capacity) {
          o_outl[at] = stash[i];
        } else {
          overflow = true;
        }
      }
    } else {
      // more outliers than the stash holds: take them from the input row in global memory again
      const uint16_t* xrow = p.x + static_cast<size_t>(tile) * p.hidden;
      unsigned long long pos = out_base;
      for (uint32_t g = 0; g < p.units; ++g) {
        const uint32_t e = 32u * g + lane;
        const uint32_t raw = e < p.hidden ? xrow[e] : 0u;
        // patterns of non-negative values order like the values; NaN patterns sort above +Inf
        const bool out = e < p.hidden && (raw & 0x7fffu) >= p.thr16;
        const uint32_t bal = __ballot_sync(kFull, out);
        if (out) {
          const unsigned long long at = pos + __popc(bal & ((1u << lane) - 1u));
          if (at < p.lay.outlier_capacity) {
            o_outl[at] = (e << 16) | raw;
          } else {
            overflow = true;
          }
        }
        pos += __popc(bal);
      }
    }
    if (__any_sync(kFull, overflow) && lane == 0) {
      atomicCAS(&p.ws->err, 0u, static_cast<uint32_t>(TSQ_ERR_OUTLIER_OVERFLOW));
    }
  }
  return TSQ_OK;
}

template <bool BF16>
__global__ void __launch_bounds__(kEncMaxWarps * 32, 1) encode_kernel(const EncodeParams p) {
  extern __shared__ __align__(128) unsigned char smem_dyn[];
  __shared__ __align__(8) uint64_t s_bar[kEncMaxWarps];

  const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
  const uint32_t gen4 = (*reinterpret_cast<volatile const uint32_t*>(&p.ws->gen) + 1u) << 2;

  if (warp < p.active_warps) {
    unsigned char* slot = smem_dyn + static_cast<size_t>(warp) * p.warp_stride;
    uint4* row = reinterpret_cast<uint4*>(slot);
    uint32_t* stash = reinterpret_cast<uint32_t*>(slot + p.row_stride);
    uint64_t* bar = &s_bar[warp];
    if (lane == 0) {
      mbar_init(bar, 1);
      mbar_fence_init();
    }
    __syncwarp();

    uint32_t parity = 0;
    bool stored = false;  // a bulk store out of the slot may still be reading it
    for (;;) {
      uint32_t tile = 0;
      if (lane == 0) tile = atomicAdd(&p.ws->ticket, 1u);
      tile = __shfl_sync(kFull, tile, 0);
      if (tile >= p.tokens) break;
      if (lane == 0) {
        if (stored) bulk_wait_read_all();
        mbar_arrive_expect_tx(bar, p.row_bytes);
        bulk_g2s(slot, p.x + static_cast<size_t>(tile) * p.hidden, p.row_bytes, bar);
      }
      stored = false;
      uint32_t err = TSQ_OK;
      if (__all_sync(kFull, mbar_wait_bounded(bar, parity, kCopyPollLimit))) {
        parity ^= 1u;
        err = encode_row<BF16>(p, gen4, tile, row, stash, lane, &stored);
      } else {
        // the copy did not land in time: tell the rows behind, give it one more bounded chance to land
        err = TSQ_ERR_TIMEOUT;
        if (lane == 0) st_relaxed_u64(p.desc + tile, pack_desc(gen4 | kFlagAbort, 0u));
        mbar_wait_bounded(bar, parity, kCopyPollLimit);
      }
      if (err != TSQ_OK) {
        if (err != 0xffffffffu && lane == 0) atomicCAS(&p.ws->err, 0u, err);
        break;
      }
      __syncwarp();  // every lane is done with the slot before the next copy overwrites it
    }
    if (lane == 0) bulk_wait_all();  // the slot must outlive the stores that read it
  }

  // ---- the CTA that finishes last publishes the status and re-arms the workspace ----
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    const uint32_t prev = atomicAdd(&p.ws->done, 1u);
    if (prev == gridDim.x - 1u) {
      __threadfence();
      const uint32_t e = atomicExch(&p.ws->err, 0u);
      // totals = the last tile's inclusive prefixes, if it got that far
      unsigned long long tw = 0ull, to = 0ull;
      if (p.tokens != 0u) {
        const unsigned long long d = ld_relaxed_u64(p.desc + (p.tokens - 1u));
        if (static_cast<uint32_t>(d >> 32) == (gen4 | kFlagPrefix)) {
          tw = static_cast<uint32_t>(d);
          __threadfence();
          to = *reinterpret_cast<volatile const uint32_t*>(p.prefix_outl + (p.tokens - 1u));
        }
      }
      write_header(p, tw, to);
      reinterpret_cast<BlobHeader*>(p.blob)->status = e;
      if (e != 0u) atomicCAS(&p.ws->enc_status, 0u, e);
      uint32_t g = (gen4 >> 2);
      if (g >= kGenWrap) {
        // generation counter about to wrap: wipe the descriptors so that old tags cannot alias
        const uint32_t n = p.ws->desc_capacity;
        for (uint32_t i = 0; i < n; ++i) p.desc[i] = 0ull;
        g = 0u;
      }
      p.ws->ticket = 0u;
      p.ws->done = 0u;
      p.ws->gen = g;
    }
  }
}

}  // namespace

cudaError_t encode_kernel_attrs(bool bf16, size_t smem) {
  const void* fn = bf16 ? reinterpret_cast<const void*>(&encode_kernel<true>)
                        : reinterpret_cast<const void*>(&encode_kernel<false>);
  return cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
}

cudaError_t launch_encode(const EncodeParams& p, int grid, int threads, size_t smem, cudaStream_t stream) {
  if (p.dtype == TSQ_BF16) {
    encode_kernel<true><<<grid, threads, smem, stream>>>(p);
  } else {
    encode_kernel<false><<<grid, threads, smem, stream>>>(p);
  }
  return cudaGetLastError();
}

}  // namespace tsq
