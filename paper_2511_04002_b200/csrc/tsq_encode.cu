// tsq encode kernel: threshold splitting (Eq. "ts") + token-wise TAB-Q (Algorithm 1 on AIQ,
// Eq. "Proposed") + bit-plane packing + CSR emission, fused into one kernel.
//
// One CTA encodes one token row, one thread per group of 32 elements (two groups per thread for
// rows longer than 32768).  A thread loads its group's 64 bytes straight into registers and the
// row never leaves them: the input is read from HBM exactly once, there is no staging copy, and
// every pass of the method is straight-line register arithmetic:
//   A  threshold split: outlier bitmap, outlier slots set to +0 (what T_below holds there), and
//      the row's min / max of the inlier magnitudes (CTA reduction);
//   B  Algorithm 1: AIQ codes at the top level and at each lower candidate, distortion sums
//      (CTA reduction, one candidate at a time, stopping at the first failure);
//   C  codes at the chosen level -> bytes (code | sign << 7) -> 8 x 32 bit transpose -> the
//      group's b* plane words, stored as one contiguous run per thread.
// The scalar work between the passes (scales, zero-points, the check described below, the
// placement) is done by warp 0 alone; the other CTAs resident on the SM fill those gaps.
//
// The binding resource is the integer / logic pipe, which issues at half the rate of the FMA pipe:
// the passes work on two 16-bit elements per 32-bit register wherever they can, and shifts and
// byte merges are written as integer multiply-adds so that they go to the FMA pipe instead.
//
// Variable-length placement: where a token's planes and CSR entries start is an exclusive prefix
// sum over all earlier tokens.  It is resolved with a decoupled look-back over per-token
// descriptors in the workspace.  Rows are numbered by an atomic ticket taken when a CTA starts,
// so a row only ever waits for rows whose CTAs are already running.  A row publishes its own
// sizes right after pass B and looks back only after pass C, so that the wait for slower
// predecessors overlaps its own packing.  A look-back step reads 256 descriptors at once (eight
// independent loads per lane).  Every wait is bounded and fails into a status word.
//
// Arithmetic contract: the codes equal  clamp(rint(m / s) - zp, 0, Qmax)  with the IEEE binary32
// quotient m / s.  Three evaluations of it exist, chosen per row:
//   kFast     rint(m * r) with r = fl(1/s), one FMA against 2^23.  It can differ from the
//             contract only when m / s lies within a relative 2^-22 of a rounding boundary k + 1/2
//             (exact ties included: 16-bit inputs make m / s land exactly on k + 1/2 quite often).
//             16-bit values are at least 2^-11 apart, so for each boundary only its two
//             neighbouring 16-bit values can be affected; those are examined per row, a cheap
//             distance test first and the true division for the few that fail it.
//   kRefined  for a row where any of them really disagrees: the correctly rounded quotient from
//             q0 = fl(m * r), the exact residual m - q0 * s (one FMA) and q = fl(q0 + residual * r)
//             (the classical FMA division step, exact when r is the correctly rounded reciprocal
//             and nothing over- or underflows), then the same 2^23 rounding.
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
  c.r = __frcp_rn(c.s);
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

// Examine every rounding boundary of every candidate level, one boundary per thread at a time
// (the levels' boundaries are numbered end to end, the top level first).
template <bool BF16>
__device__ __forceinline__ bool any_boundary_disagrees(const Level* lv, int n_levels, uint32_t pmin, uint32_t pmax,
                                                       uint32_t tid, uint32_t nthreads) {
  int total = 0;
  for (int i = 0; i < n_levels; ++i) total += lv[i].qmax + 2;
  bool bad = false;
  for (int t = static_cast<int>(tid); t < total; t += static_cast<int>(nthreads)) {
    int i = n_levels - 1, j = t;
    while (j >= lv[i].qmax + 2) {
      j -= lv[i].qmax + 2;
      --i;
    }
    bad |= boundary_disagrees<BF16>(lv[i], j, pmin, pmax);
  }
  return bad;
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

// Pass B on one group: sum |(q0 >> sh) - q| over its 32 elements (Algorithm 1's distortion numerator).
template <bool BF16, int MODE>
__device__ __forceinline__ uint32_t distortion_group(const uint32_t (&x)[16], const Level& top, const Level& low,
                                                     int sh) {
  const uint32_t shmask = (0xffffu >> sh) * 0x10001u;
  uint32_t S2 = 0;  // two 16-bit partial sums: at most 16 * 127 each
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    const uint32_t a = (codes2<BF16, MODE>(x[i], top) >> sh) & shmask;
    const uint32_t q = codes2<BF16, MODE>(x[i], low);
    S2 += max_s16x2(a, q) - min_s16x2(a, q);
  }
  return (S2 & 0xffffu) + (S2 >> 16);
}

// Pass C on one group: codes at the chosen level as bytes (code | sign << 7), transposed into
// bit-planes: on return r[k] = bit k of every byte, k < 7 code bits, k = 7 signs.
template <bool BF16, int MODE>
__device__ __forceinline__ void pack_group(const uint32_t (&x)[16], const Level& lv, uint32_t (&r)[8]) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    // b2 of chunk j: bytes of elements 8j + 2i (byte 0) and 8j + 2i + 1 (byte 2)
    uint32_t b2[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) b2[j] = codes2<BF16, MODE>(x[4 * j + i], lv) | ((x[4 * j + i] >> 8) & 0x00800080u);
    const uint32_t e = b2[1] * 256u + b2[0];  // bytes: elements 2i, 8 + 2i, 2i + 1, 8 + 2i + 1
    const uint32_t f = b2[3] * 256u + b2[2];  // the same, 16 further on
    r[2 * i] = __byte_perm(e, f, 0x5410);      // byte c = element 8c + 2i
    r[2 * i + 1] = __byte_perm(e, f, 0x7632);  // byte c = element 8c + 2i + 1
  }
  transpose8x32(r);
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
__device__ int resolve_prefix(const EncodeParams& p, uint32_t gen4, uint32_t tile, uint32_t agg_w, uint32_t agg_o,
                              uint32_t lane, uint32_t* excl_w, uint32_t* excl_o) {
  uint32_t base_w = 0, base_o = 0;  // prefix found at the end of the walk
  uint32_t part_w = 0, part_o = 0;  // this lane's share of the aggregates walked over
  if (tile > 0) {
    int pos = static_cast<int>(tile) - 1;  // nearest tile not yet accounted for
    uint32_t polls = 0;
    bool done = false;
    while (!done) {
      unsigned long long vw[kLookbackDepth], vo[kLookbackDepth];
#pragma unroll
      for (int k = 0; k < kLookbackDepth; ++k) {
        const int j = pos - (32 * k + static_cast<int>(lane));
        // before tile 0: prefix 0
        vw[k] = j >= 0 ? ld_relaxed_u64(p.desc + 2 * static_cast<size_t>(j)) : pack_desc(gen4 | kFlagPrefix, 0u);
        vo[k] = j >= 0 ? ld_relaxed_u64(p.desc + 2 * static_cast<size_t>(j) + 1) : pack_desc(gen4 | kFlagPrefix, 0u);
      }
      int consumed = 32 * kLookbackDepth;
      bool stopped = false;
      int verdict = TSQ_OK;
#pragma unroll
      for (int k = 0; k < kLookbackDepth; ++k) {
        if (stopped) continue;
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
          if (++polls > kLookbackPollLimit) return TSQ_ERR_TIMEOUT;
          __nanosleep(polls < 16u ? 100u : 500u);
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
  for (int i = 0; i < 8; ++i) h->bits[i] = (i < p.n_bits) ? static_cast<uint8_t>(p.bits[i]) : 0;
  h->tau = p.tau;
  h->delta = p.delta;
  h->total_words = total_words;
  h->total_outliers = total_outliers;
  h->outlier_capacity = static_cast<uint32_t>(p.lay.outlier_capacity);
}

// What the CTA shares about its row.
struct RowShared {
  Level lv[kMaxCand];  // lv[i]: AIQ parameters of candidate bits[i]
  int S[kMaxCand];     // distortion sum of candidate i against the top level
  uint32_t tile;
  int mode;            // kFast or kDivide from the scales alone; kFast becomes kRefined when `bad` is set
  uint32_t bad;        // some boundary of some level is not safe for the one-FMA path
  uint32_t pmin, pmax; // patterns of the row's smallest and largest inlier magnitude
  uint32_t row_cnt;    // outliers of the row
  uint32_t word_off, out_base;
  uint32_t status;     // TSQ_OK, or why the row is not written
  uint32_t warp_min[32], warp_max[32], warp_cnt[32];  // per-warp partial results; warp_cnt becomes an exclusive scan
};

template <bool BF16, int UPT>
__global__ void __launch_bounds__(1024, 1) encode_kernel(const EncodeParams p) {
  using E = Elem<BF16>;
  __shared__ RowShared sh;
  const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5, nwarps = blockDim.x >> 5;
  const uint32_t gen4 = (*reinterpret_cast<volatile const uint32_t*>(&p.ws->gen) + 1u) << 2;

  if (tid == 0) {
    sh.tile = atomicAdd(&p.ws->ticket, 1u);
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
    {
      const uint32_t mnv = __reduce_min_sync(kFull, min(mn2 & 0xffffu, mn2 >> 16));
      const uint32_t mxv = __reduce_max_sync(kFull, max(mx2 & 0xffffu, mx2 >> 16));
      const uint32_t wcnt = __reduce_add_sync(kFull, cnt);
      if (lane == 0) {
        sh.warp_min[warp] = mnv;
        sh.warp_max[warp] = mxv;
        sh.warp_cnt[warp] = wcnt;
      }
    }
    __syncthreads();

    // ---- AIQ parameters of every candidate level (lane i of warp 0 takes candidate i) ----
    const int bmax = p.bits[p.n_bits - 1];
    if (warp == 0) {
      const uint32_t pmin = __reduce_min_sync(kFull, lane < nwarps ? sh.warp_min[lane] : 0xffffu);
      const uint32_t pmax = __reduce_max_sync(kFull, lane < nwarps ? sh.warp_max[lane] : 0u);
      // exclusive scan of the per-warp outlier counts
      const uint32_t wc = lane < nwarps ? sh.warp_cnt[lane] : 0u;
      uint32_t incl = wc;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const uint32_t n = __shfl_up_sync(kFull, incl, d);
        if (lane >= static_cast<uint32_t>(d)) incl += n;
      }
      sh.warp_cnt[lane] = incl - wc;
      const uint32_t total = __shfl_sync(kFull, incl, 31);
      const Level lv = make_level(E::pattern_f32(pmin), E::pattern_f32(pmax), p.bits[min(lane, static_cast<uint32_t>(p.n_bits - 1))]);
      if (lane < static_cast<uint32_t>(p.n_bits)) {
        sh.lv[lane] = lv;
        sh.S[lane] = 0;
      }
      const bool all_fast = __all_sync(kFull, lv.fast);
      if (lane == 0) {
        sh.mode = all_fast ? kFast : kDivide;
        sh.bad = 0u;
        sh.pmin = pmin;
        sh.pmax = pmax;
        sh.row_cnt = total;
      }
    }
    __syncthreads();
    // ---- may the one-FMA path be trusted for this row?  every boundary of every level, all threads ----
    if (sh.mode == kFast) {
      if (any_boundary_disagrees<BF16>(sh.lv, p.n_bits, sh.pmin, sh.pmax, tid, blockDim.x)) sh.bad = 1u;
      __syncthreads();
    }
    const int mode = (sh.mode == kFast && sh.bad != 0u) ? kRefined : sh.mode;

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
        S += mode == kFast      ? distortion_group<BF16, kFast>(x[k], top, low, shn)
             : mode == kRefined ? distortion_group<BF16, kRefined>(x[k], top, low, shn)
                                : distortion_group<BF16, kDivide>(x[k], top, low, shn);
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
      if (mode == kFast) {
        pack_group<BF16, kFast>(x[k], best, r[k]);
      } else if (mode == kRefined) {
        pack_group<BF16, kRefined>(x[k], best, r[k]);
      } else {
        pack_group<BF16, kDivide>(x[k], best, r[k]);
      }
    }

    // ---- placement: exclusive prefix sums over the tokens before this one ----
    if (warp == 0) {
      uint32_t word_off = 0, out_base = 0;
      const int st = resolve_prefix(p, gen4, tile, agg_w, row_cnt, lane, &word_off, &out_base);
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
      // ---- plane words: group u owns words u * b* .. u * b* + b* - 1, plane 0 = sign, plane 1 + k = code bit k ----
      uint32_t* wrow = reinterpret_cast<uint32_t*>(p.blob + p.lay.off_words) + word_off;
#pragma unroll
      for (int k = 0; k < UPT; ++k) {
        const uint32_t u = UPT * tid + k;
        if (u >= p.units) continue;
        uint32_t* dst = wrow + static_cast<size_t>(u) * bstar;
        if (p.vec_store && bstar == 8) {
          reinterpret_cast<uint4*>(dst)[0] = make_uint4(r[k][7], r[k][0], r[k][1], r[k][2]);
          reinterpret_cast<uint4*>(dst)[1] = make_uint4(r[k][3], r[k][4], r[k][5], r[k][6]);
        } else if (p.vec_store && bstar == 4) {
          reinterpret_cast<uint4*>(dst)[0] = make_uint4(r[k][7], r[k][0], r[k][1], r[k][2]);
        } else {
          dst[0] = r[k][7];
#pragma unroll
          for (int q = 0; q < 7; ++q) {
            if (q < bstar - 1) dst[1 + q] = r[k][q];
          }
        }
      }
      if (tid == 0) {
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
          unsigned long long at = static_cast<unsigned long long>(out_base) + sh.warp_cnt[warp] + (incl - cnt);
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

  // ---- the CTA that finishes last publishes the status and re-arms the workspace ----
  __syncthreads();
  if (tid == 0) {
    __threadfence();
    const uint32_t prev = atomicAdd(&p.ws->done, 1u);
    if (prev == gridDim.x - 1u) {
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
  }
}

}  // namespace

cudaError_t launch_encode(const EncodeParams& p, int grid, int threads, int upt, cudaStream_t stream) {
  const bool bf16 = p.dtype == TSQ_BF16;
  if (upt == 1) {
    if (bf16) {
      encode_kernel<true, 1><<<grid, threads, 0, stream>>>(p);
    } else {
      encode_kernel<false, 1><<<grid, threads, 0, stream>>>(p);
    }
  } else {
    if (bf16) {
      encode_kernel<true, 2><<<grid, threads, 0, stream>>>(p);
    } else {
      encode_kernel<false, 2><<<grid, threads, 0, stream>>>(p);
    }
  }
  return cudaGetLastError();
}

}  // namespace tsq
