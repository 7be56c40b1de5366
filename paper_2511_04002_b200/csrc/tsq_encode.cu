// tsq encode kernel: threshold splitting (Eq. "ts") + token-wise TAB-Q (Algorithm 1 on AIQ,
// Eq. "Proposed") + bit-plane packing + CSR emission, fused into one persistent kernel.
//
// One CTA works on one token row at a time.  Rows arrive in shared memory through a ring of bulk
// asynchronous copies (one elected thread issues them, an mbarrier per stage reports the bytes),
// so the input is read from HBM exactly once.  Tiles are handed out by an atomic ticket, which
// makes the cross-CTA prefix sums (where a token's planes and CSR entries start) safe to resolve
// with a decoupled look-back: a tile only ever waits for lower tiles, and those belong to CTAs
// that are already running.  Every wait is bounded and fails into a status word.
//
// Arithmetic contract: the codes equal  clamp(rint(m / s) - zp, 0, Qmax)  with the IEEE binary32
// quotient m / s.  The fast path evaluates rint(m * r) with r = fl(1/s) in one FMA against
// 1.5 * 2^23; this can differ from the contract only for a 16-bit value that lies within 2^-22
// (relative) of a rounding boundary (k + 1/2) * s, and 16-bit values are at least 2^-11 apart,
// so for each boundary only its two neighbouring 16-bit values can be affected.  Those are
// tested explicitly per row, with the true division, and a row where any of them disagrees is
// redone entirely with true divisions.

#include "tsq_device.cuh"
#include "tsq_internal.h"

namespace tsq {
namespace {

constexpr float kRoundMagic = 12582912.0f;  // 1.5 * 2^23: adding it rounds to an integer, ties to even
constexpr int kRoundMagicBits = 0x4B400000;
constexpr uint32_t kLookbackPollLimit = 1u << 20;
constexpr uint32_t kCopyPollLimit = 1u << 20;

// AIQ parameters of one candidate level for one row (Eq. "Proposed").
struct Level {
  float s;    // scale
  float r;    // fl(1 / s), fast path only
  int zp;     // zero-point rint(m_min / s)
  int qmax;   // 2^(b-1) - 1
  bool fast;  // scale in the range where the FMA path is provably safe
};

__device__ __forceinline__ Level make_level(float mmin, float mmax, int b) {
  Level c;
  c.qmax = (1 << (b - 1)) - 1;
  const float range = __fsub_rn(mmax, mmin);
  c.s = range > 0.0f ? __fdiv_rn(range, static_cast<float>(c.qmax)) : (mmax > 0.0f ? mmax : 1.0f);
  c.zp = __float2int_rn(__fdiv_rn(mmin, c.s));
  c.r = __fdiv_rn(1.0f, c.s);
  c.fast = (c.s >= 0x1p-100f) && (c.s <= 0x1p100f);
  return c;
}

template <bool EXACT>
__device__ __forceinline__ int code_of(float m, const Level& c) {
  int k;
  if (EXACT) {
    k = __float2int_rn(__fdiv_rn(m, c.s)) - c.zp;
  } else {
    k = __float_as_int(fmaf(m, c.r, kRoundMagic)) - kRoundMagicBits - c.zp;
  }
  return min(max(k, 0), c.qmax);
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
  bool bad = false;
#pragma unroll
  for (uint32_t d = 0; d < 2; ++d) {
    const uint32_t pat = plo + d;
    if (pat >= pmin && pat <= pmax) {
      const float m = E::pattern_f32(pat);
      bad |= code_of<false>(m, c) != code_of<true>(m, c);
    }
  }
  return bad;
}

// Numerator of Algorithm 1's distortion for this thread's units: sum |(q0 >> sh) - q|.
template <bool BF16, bool EXACT>
__device__ __forceinline__ int distortion_partial(const uint4* row, const EncodeParams& p, uint32_t thr2,
                                                  const Level& top, const Level& low, int sh) {
  using E = Elem<BF16>;
  int S = 0;
  for (uint32_t u = threadIdx.x; u < p.units; u += blockDim.x) {
    const uint32_t rot = (u >> 1) & 3u;
#pragma unroll
    for (uint32_t j = 0; j < 4; ++j) {
      const uint32_t cidx = 4u * u + ((j + rot) & 3u);
      if (cidx >= p.chunks) continue;
      const uint4 c = row[cidx];
      const uint32_t x[4] = {c.x, c.y, c.z, c.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t a = x[i] & 0x7fff7fffu;
        const uint32_t m2 = a & ~E::geu_mask(a, thr2);
        const float mlo = E::lo_f32(m2), mhi = E::hi_f32(m2);
        S += abs((code_of<EXACT>(mlo, top) >> sh) - code_of<EXACT>(mlo, low));
        S += abs((code_of<EXACT>(mhi, top) >> sh) - code_of<EXACT>(mhi, low));
      }
    }
  }
  return S;
}

// Codes of one unit at the chosen level, packed as bytes (code << 1 | sign), transposed into
// bit-planes and stored: plane 0 = sign, plane 1 + k = bit k of the code.
template <bool BF16, bool EXACT>
__device__ __forceinline__ void pack_units(const uint4* row, const EncodeParams& p, uint32_t thr2, const Level& lv,
                                           int bstar, uint32_t* wdst) {
  using E = Elem<BF16>;
  for (uint32_t u = threadIdx.x; u < p.units; u += blockDim.x) {
    const uint32_t rot = (u >> 1) & 3u;
    uint32_t r[8] = {0, 0, 0, 0, 0, 0, 0, 0};
#pragma unroll
    for (uint32_t j = 0; j < 4; ++j) {
      const uint32_t cc = (j + rot) & 3u;
      const uint32_t cidx = 4u * u + cc;
      if (cidx >= p.chunks) continue;
      const uint4 c = row[cidx];
      const uint32_t x[4] = {c.x, c.y, c.z, c.w};
      const uint32_t shift = 8u * cc;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t a = x[i] & 0x7fff7fffu;
        const uint32_t mk = E::geu_mask(a, thr2);
        const uint32_t keep = x[i] & ~mk;  // inliers keep sign and magnitude, outlier slots become +0
        const uint32_t m2 = keep & 0x7fff7fffu;
        const uint32_t blo = (static_cast<uint32_t>(code_of<EXACT>(E::lo_f32(m2), lv)) << 1) | ((keep >> 15) & 1u);
        const uint32_t bhi = (static_cast<uint32_t>(code_of<EXACT>(E::hi_f32(m2), lv)) << 1) | (keep >> 31);
        r[2 * i] |= blo << shift;
        r[2 * i + 1] |= bhi << shift;
      }
    }
    transpose8x32(r);
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      if (k < bstar) wdst[static_cast<size_t>(k) * p.lay.wpp + u] = r[k];
    }
  }
}

__device__ __forceinline__ unsigned long long pack_desc(uint32_t tag, uint32_t value) {
  return (static_cast<unsigned long long>(tag) << 32) | value;
}

// Decoupled look-back over the tile descriptors, run by one full warp.  Publishes this tile's
// aggregates, sums the predecessors' contributions until an inclusive prefix is met, then
// publishes this tile's inclusive prefixes.  Returns TSQ_OK, TSQ_ERR_TIMEOUT (gave up) or
// a value < 0 when a predecessor has aborted.
__device__ int lookback(const EncodeParams& p, uint32_t gen4, uint32_t tile, uint32_t agg_w, uint32_t agg_o,
                        uint32_t* excl_w, uint32_t* excl_o) {
  const uint32_t lane = threadIdx.x & 31u;
  uint32_t sum_w = 0, sum_o = 0;
  if (tile > 0) {
    if (lane == 0) {
      st_relaxed_u64(p.desc_words + tile, pack_desc(gen4 | kFlagAggregate, agg_w));
      st_relaxed_u64(p.desc_outl + tile, pack_desc(gen4 | kFlagAggregate, agg_o));
    }
    bool done_w = false, done_o = false;
    uint32_t polls = 0;
    for (int base = static_cast<int>(tile) - 1; !(done_w && done_o); base -= 32) {
      const int j = base - static_cast<int>(lane);
      const bool valid = j >= 0;
      unsigned long long vw = 0, vo = 0;
      uint32_t fw = 0, fo = 0;
      for (;;) {
        if (valid) {
          vw = ld_relaxed_u64(p.desc_words + j);
          vo = ld_relaxed_u64(p.desc_outl + j);
        }
        const uint32_t tw = static_cast<uint32_t>(vw >> 32), to = static_cast<uint32_t>(vo >> 32);
        fw = ((tw & ~3u) == gen4) ? (tw & 3u) : 0u;
        fo = ((to & ~3u) == gen4) ? (to & 3u) : 0u;
        if (__all_sync(kFull, !valid || (fw != 0u && fo != 0u))) break;
        if (++polls > kLookbackPollLimit) return TSQ_ERR_TIMEOUT;
        __nanosleep(40);
      }
      if (__any_sync(kFull, valid && (fw == kFlagAbort || fo == kFlagAbort))) return -1;
      const uint32_t before_start = __ballot_sync(kFull, !valid);  // lanes that fell off tile 0: the chain ends there
      if (!done_w) {
        const uint32_t stop = __ballot_sync(kFull, valid && fw == kFlagPrefix) | before_start;
        const uint32_t first = stop ? static_cast<uint32_t>(__ffs(stop) - 1) : 32u;
        sum_w += __reduce_add_sync(kFull, (valid && lane <= first) ? static_cast<uint32_t>(vw) : 0u);
        done_w = stop != 0u;
      }
      if (!done_o) {
        const uint32_t stop = __ballot_sync(kFull, valid && fo == kFlagPrefix) | before_start;
        const uint32_t first = stop ? static_cast<uint32_t>(__ffs(stop) - 1) : 32u;
        sum_o += __reduce_add_sync(kFull, (valid && lane <= first) ? static_cast<uint32_t>(vo) : 0u);
        done_o = stop != 0u;
      }
    }
  }
  if (lane == 0) {
    st_relaxed_u64(p.desc_words + tile, pack_desc(gen4 | kFlagPrefix, sum_w + agg_w));
    st_relaxed_u64(p.desc_outl + tile, pack_desc(gen4 | kFlagPrefix, sum_o + agg_o));
  }
  *excl_w = sum_w;
  *excl_o = sum_o;
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

template <bool BF16>
__global__ void __launch_bounds__(kMaxThreads) encode_kernel(const EncodeParams p) {
  using E = Elem<BF16>;
  extern __shared__ __align__(128) unsigned char smem_dyn[];
  __shared__ __align__(8) uint64_t s_bar[kMaxStages];
  __shared__ uint32_t s_tile[kMaxStages];
  __shared__ uint32_t s_red_a[8][4];
  __shared__ int s_red_b[2][8][2];
  __shared__ uint32_t s_lb[4];

  const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5, nwarps = blockDim.x >> 5;
  const uint32_t row_stride = (p.row_bytes + 127u) & ~127u;
  uint32_t* s_ucnt = reinterpret_cast<uint32_t*>(smem_dyn + static_cast<size_t>(p.stages) * row_stride);
  const uint32_t gen4 = (*reinterpret_cast<volatile const uint32_t*>(&p.ws->gen) + 1u) << 2;
  const uint32_t thr2 = p.thr16 * 0x10001u;

  uint32_t* o_word_off = reinterpret_cast<uint32_t*>(p.blob + p.lay.off_word_off);
  uint32_t* o_out_ptr = reinterpret_cast<uint32_t*>(p.blob + p.lay.off_out_ptr);
  uint32_t* o_words = reinterpret_cast<uint32_t*>(p.blob + p.lay.off_words);
  uint32_t* o_outl = reinterpret_cast<uint32_t*>(p.blob + p.lay.off_outl);

  uint32_t issued[kMaxStages] = {0, 0, 0, 0};  // thread 0: copies issued per stage
  uint32_t pending = 0;                        // thread 0: stages with a copy not yet consumed

  if (tid == 0) {
    for (uint32_t s = 0; s < p.stages; ++s) mbar_init(&s_bar[s], 1);
    mbar_fence_init();
  }
  __syncthreads();
  if (tid == 0) {
    for (uint32_t s = 0; s < p.stages; ++s) {
      const uint32_t t = atomicAdd(&p.ws->ticket, 1u);
      s_tile[s] = t;
      if (t < p.tokens) {
        mbar_arrive_expect_tx(&s_bar[s], p.row_bytes);
        bulk_g2s(smem_dyn + static_cast<size_t>(s) * row_stride, p.x + static_cast<size_t>(t) * p.hidden, p.row_bytes,
                 &s_bar[s]);
        issued[s] = 1;
        pending |= 1u << s;
      }
    }
  }
  __syncthreads();

  uint32_t err = TSQ_OK;
  uint32_t rb = 0;  // which half of s_red_b the next reduction uses
  uint32_t cur_tile = 0xffffffffu;

  for (uint32_t it = 0;; ++it) {
    const uint32_t stage = it % p.stages;
    const uint32_t parity = (it / p.stages) & 1u;
    const uint32_t tile = s_tile[stage];
    if (tile >= p.tokens) break;
    cur_tile = tile;
    const uint4* row = reinterpret_cast<const uint4*>(smem_dyn + static_cast<size_t>(stage) * row_stride);
    const bool arrived = mbar_wait_bounded(&s_bar[stage], parity, kCopyPollLimit);
    if (tid == 0 && arrived) pending &= ~(1u << stage);

    // ---- pass A: threshold split, per-token min / max of the magnitudes, outlier counts ----
    uint32_t mn2 = E::kInfPattern * 0x10001u, mx2 = 0u, cnt = 0u;
    if (arrived) {
      for (uint32_t u = tid; u < p.units; u += blockDim.x) {
        const uint32_t rot = (u >> 1) & 3u;
        uint32_t any = 0u;
#pragma unroll
        for (uint32_t j = 0; j < 4; ++j) {
          const uint32_t cidx = 4u * u + ((j + rot) & 3u);
          if (cidx >= p.chunks) continue;
          const uint4 c = row[cidx];
          const uint32_t x[4] = {c.x, c.y, c.z, c.w};
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const uint32_t a = x[i] & 0x7fff7fffu;
            const uint32_t mk = E::geu_mask(a, thr2);
            const uint32_t m2 = a & ~mk;
            mx2 = E::max2(mx2, m2);
            mn2 = E::min2(mn2, m2);
            any |= mk;
          }
        }
        uint32_t ucount = 0u;
        if (any) {
          for (uint32_t j = 0; j < 4; ++j) {
            const uint32_t cidx = 4u * u + j;
            if (cidx >= p.chunks) continue;
            const uint4 c = row[cidx];
            const uint32_t x[4] = {c.x, c.y, c.z, c.w};
            for (int i = 0; i < 4; ++i) ucount += __popc(E::geu_mask(x[i] & 0x7fff7fffu, thr2));
          }
          ucount >>= 4;
        }
        s_ucnt[u] = ucount;
        cnt += ucount;
      }
    }
    {
      uint32_t mnv = min(mn2 & 0xffffu, mn2 >> 16), mxv = max(mx2 & 0xffffu, mx2 >> 16);
      mnv = __reduce_min_sync(kFull, mnv);
      mxv = __reduce_max_sync(kFull, mxv);
      cnt = __reduce_add_sync(kFull, cnt);
      const uint32_t okw = __all_sync(kFull, arrived) ? 1u : 0u;
      if (lane == 0) {
        s_red_a[warp][0] = mnv;
        s_red_a[warp][1] = mxv;
        s_red_a[warp][2] = cnt;
        s_red_a[warp][3] = okw;
      }
    }
    __syncthreads();
    uint32_t pmin = 0xffffu, pmax = 0u, row_cnt = 0u, all_ok = 1u;
    for (uint32_t w = 0; w < nwarps; ++w) {
      pmin = min(pmin, s_red_a[w][0]);
      pmax = max(pmax, s_red_a[w][1]);
      row_cnt += s_red_a[w][2];
      all_ok &= s_red_a[w][3];
    }
    if (!all_ok) {
      err = TSQ_ERR_TIMEOUT;
      break;
    }

    // ---- Algorithm 1: descend the candidate list while the distortion stays within tolerance ----
    const float mmin = E::pattern_f32(pmin), mmax = E::pattern_f32(pmax);
    const int bmax = p.bits[p.n_bits - 1];
    const Level top = make_level(mmin, mmax, bmax);
    Level best = top;
    int bstar = bmax;
    bool exact = !top.fast;  // once set, the whole row is evaluated with true divisions
    bool top_checked = false;
    if (p.n_bits == 1 && !exact) {
      bool bad = false;
      for (int j = tid; j <= top.qmax + 1; j += blockDim.x) bad |= boundary_disagrees<BF16>(top, j, pmin, pmax);
      exact = __syncthreads_or(bad) != 0;
    }
    for (int ci = p.n_bits - 2; ci >= 0; --ci) {
      const int b = p.bits[ci];
      const Level low = make_level(mmin, mmax, b);
      const int sh = bmax - b;
      if (!low.fast) exact = true;
      int S_total = 0;
      for (;;) {
        int S;
        uint32_t bad = 0u;
        if (exact) {
          S = distortion_partial<BF16, true>(row, p, thr2, top, low, sh);
        } else {
          S = distortion_partial<BF16, false>(row, p, thr2, top, low, sh);
          const int n_top = top_checked ? 0 : top.qmax + 2;
          const int n_items = n_top + low.qmax + 2;
          for (int w = tid; w < n_items; w += blockDim.x) {
            bad |= (w < n_top) ? boundary_disagrees<BF16>(top, w, pmin, pmax)
                               : boundary_disagrees<BF16>(low, w - n_top, pmin, pmax);
          }
        }
        S = __reduce_add_sync(kFull, S);
        bad = __any_sync(kFull, bad) ? 1u : 0u;
        if (lane == 0) {
          s_red_b[rb][warp][0] = S;
          s_red_b[rb][warp][1] = static_cast<int>(bad);
        }
        __syncthreads();
        S_total = 0;
        int bad_total = 0;
        for (uint32_t w = 0; w < nwarps; ++w) {
          S_total += s_red_b[rb][w][0];
          bad_total |= s_red_b[rb][w][1];
        }
        rb ^= 1u;
        if (!exact && bad_total) {
          exact = true;  // redo this level, and everything after it, with true divisions
          continue;
        }
        break;
      }
      top_checked = true;
      if (S_total > p.s_max) break;  // delta > Delta: keep the last level that passed
      bstar = b;
      best = low;
    }

    // ---- placement: exclusive prefix sums over the tokens before this one ----
    if (warp == 0) {
      uint32_t excl_w = 0, excl_o = 0;
      const int st = lookback(p, gen4, tile, static_cast<uint32_t>(bstar) * p.lay.wpp, row_cnt, &excl_w, &excl_o);
      if (st == TSQ_OK) {
        if (row_cnt != 0u) {
          // exclusive scan of the per-unit outlier counts, in place; s_ucnt[units] = row total
          uint32_t carry = 0;
          for (uint32_t base = 0; base < p.units; base += 32) {
            const uint32_t u = base + lane;
            const uint32_t v = (u < p.units) ? s_ucnt[u] : 0u;
            uint32_t incl = v;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
              const uint32_t n = __shfl_up_sync(kFull, incl, d);
              if (lane >= static_cast<uint32_t>(d)) incl += n;
            }
            if (u < p.units) s_ucnt[u] = carry + incl - v;
            carry += __shfl_sync(kFull, incl, 31);
          }
          if (lane == 0) s_ucnt[p.units] = carry;
        }
        if (lane == 0) {
          reinterpret_cast<uint8_t*>(p.blob + p.lay.off_bits)[tile] = static_cast<uint8_t>(bstar);
          reinterpret_cast<float*>(p.blob + p.lay.off_scale)[tile] = best.s;
          reinterpret_cast<int32_t*>(p.blob + p.lay.off_zp)[tile] = best.zp;
          if (tile == 0) {
            o_word_off[0] = 0;
            o_out_ptr[0] = 0;
          }
          const uint32_t incl_w = excl_w + static_cast<uint32_t>(bstar) * p.lay.wpp;
          const uint32_t incl_o = excl_o + row_cnt;
          o_word_off[tile + 1] = incl_w;
          o_out_ptr[tile + 1] = incl_o;
        }
      }
      if (lane == 0) {
        s_lb[0] = excl_w;
        s_lb[1] = excl_o;
        s_lb[2] = static_cast<uint32_t>(st == TSQ_OK ? 0 : (st < 0 ? 0xffffffffu : static_cast<uint32_t>(st)));
      }
    }
    __syncthreads();
    if (s_lb[2] != 0u) {
      err = (s_lb[2] == 0xffffffffu) ? 0xffffffffu : s_lb[2];
      break;
    }
    const uint32_t word_off = s_lb[0], out_base = s_lb[1];

    // ---- pack the planes of the chosen level ----
    if (exact) {
      pack_units<BF16, true>(row, p, thr2, best, bstar, o_words + word_off);
    } else {
      pack_units<BF16, false>(row, p, thr2, best, bstar, o_words + word_off);
    }

    // ---- CSR entries of T_above: ascending columns, original patterns ----
    if (row_cnt != 0u) {
      const uint16_t* row16 = reinterpret_cast<const uint16_t*>(row);
      bool overflow = false;
      for (uint32_t u = tid; u < p.units; u += blockDim.x) {
        const uint32_t first = s_ucnt[u], n = s_ucnt[u + 1] - first;
        if (n == 0u) continue;
        unsigned long long pos = static_cast<unsigned long long>(out_base) + first;
        const uint32_t e_end = min(32u * u + 32u, p.hidden);
        for (uint32_t e = 32u * u; e < e_end; ++e) {
          const uint32_t raw = row16[e];
          const bool out = (raw & 0x7fffu) >= p.thr16;  // patterns of non-negative values order like the values; NaN sorts last
          if (out) {
            if (pos < p.lay.outlier_capacity) {
              o_outl[pos] = (e << 16) | raw;
            } else {
              overflow = true;
            }
            ++pos;
          }
        }
      }
      if (overflow) atomicCAS(&p.ws->err, 0u, static_cast<uint32_t>(TSQ_ERR_OUTLIER_OVERFLOW));
    }

    // ---- hand the stage back and fetch the next row into it ----
    __syncthreads();
    if (tid == 0) {
      const uint32_t t = atomicAdd(&p.ws->ticket, 1u);
      s_tile[stage] = t;
      if (t < p.tokens) {
        mbar_arrive_expect_tx(&s_bar[stage], p.row_bytes);
        bulk_g2s(smem_dyn + static_cast<size_t>(stage) * row_stride, p.x + static_cast<size_t>(t) * p.hidden,
                 p.row_bytes, &s_bar[stage]);
        issued[stage] += 1;
        pending |= 1u << stage;
      }
    }
    // s_tile[stage] is next read `stages` iterations from now, several barriers later,
    // except with a single stage, where the very next iteration reads it.
    if (p.stages == 1u) __syncthreads();
  }

  // ---- abort path: tell the tiles behind us, then let copies in flight land ----
  if (err != TSQ_OK && tid == 0) {
    if (err != 0xffffffffu) atomicCAS(&p.ws->err, 0u, err);
    for (uint32_t s = 0; s < p.stages; ++s) {
      const uint32_t t = s_tile[s];
      if (t < p.tokens && t >= cur_tile) {
        st_relaxed_u64(p.desc_words + t, pack_desc(gen4 | kFlagAbort, 0u));
        st_relaxed_u64(p.desc_outl + t, pack_desc(gen4 | kFlagAbort, 0u));
      }
    }
    for (uint32_t s = 0; s < p.stages; ++s) {
      if (pending & (1u << s)) mbar_wait_bounded(&s_bar[s], (issued[s] - 1u) & 1u, kCopyPollLimit);
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
        const unsigned long long dw = ld_relaxed_u64(p.desc_words + (p.tokens - 1u));
        const unsigned long long dout = ld_relaxed_u64(p.desc_outl + (p.tokens - 1u));
        if (static_cast<uint32_t>(dw >> 32) == (gen4 | kFlagPrefix)) tw = static_cast<uint32_t>(dw);
        if (static_cast<uint32_t>(dout >> 32) == (gen4 | kFlagPrefix)) to = static_cast<uint32_t>(dout);
      }
      write_header(p, tw, to);
      reinterpret_cast<BlobHeader*>(p.blob)->status = e;
      if (e != 0u) atomicCAS(&p.ws->enc_status, 0u, e);
      uint32_t g = (gen4 >> 2);
      if (g >= kGenWrap) {
        // generation counter about to wrap: wipe the descriptors so that old tags cannot alias
        const uint32_t n = p.ws->desc_capacity;
        for (uint32_t i = 0; i < n; ++i) {
          p.desc_words[i] = 0ull;
          p.desc_outl[i] = 0ull;
        }
        g = 0u;
      }
      p.ws->ticket = 0u;
      p.ws->done = 0u;
      p.ws->gen = g;
    }
  }
}

}  // namespace

size_t encode_smem_bytes(uint32_t units, uint32_t row_bytes, uint32_t stages) {
  const size_t row_stride = (static_cast<size_t>(row_bytes) + 127u) & ~static_cast<size_t>(127u);
  return stages * row_stride + (static_cast<size_t>(units) + 1u) * sizeof(uint32_t);
}

cudaError_t encode_kernel_attrs(bool bf16, int threads, size_t smem, int* blocks_per_sm) {
  const void* fn = bf16 ? reinterpret_cast<const void*>(&encode_kernel<true>)
                        : reinterpret_cast<const void*>(&encode_kernel<false>);
  cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (e != cudaSuccess) return e;
  return cudaOccupancyMaxActiveBlocksPerMultiprocessor(blocks_per_sm, fn, threads, smem);
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
