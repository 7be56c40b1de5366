// tsq_ref — CPU oracle for threshold splitting (TS) + token-wise adaptive bit
// quantisation (TAB-Q), encode and decode.
//
// THIS FILE IS TEST INFRASTRUCTURE.  It is the slow, plain, single-threaded
// statement of what the codec computes, written from the paper's equations and
// Algorithm 1.  It shares no code, header, table or constant with the CUDA
// library and must never be called from the product path; only the test-suite,
// the smoke check and the benchmark's CPU-baseline leg may load it.
//
// Build: g++ -std=c++17 -O2 -ffp-contract=off -fno-fast-math -shared -fPIC
// (IEEE binary32, round-to-nearest-even, no FMA contraction, no flush-to-zero).
//
// What is computed, per token row (H raw 16-bit patterns), and where the paper
// defines it:
//   * TS (Eq. "ts"):  M_j = 1 iff |T_j| >= tau.  T_above goes, undistorted, to a
//     CSR list (Sec. II-C.1); T_below = T*(1-M) keeps a +0 in every outlier slot.
//   * TAB-Q (Algorithm 1, applied token-wise, Sec. II-C.2): sign and magnitude
//     are separated (lines 1-2); the magnitudes are quantised by AIQ
//     (Eq. "Proposed") at the highest level, then at each lower candidate level,
//     with distortion  delta = sum | floor(T0 / 2^(Qbar-Q)) - T^ | / n  compared
//     against the tolerance Delta (lines 5-14).
//   * Restore (Eq. "dequnt"):  T~ = (code, zero-point) * scale  + T_above.
//
// Readings taken where the paper is silent, garbled or at odds with itself
// (each is restated in the design notes of this repository):
//   R1  zero-point sign: Eq. "Proposed" adds z while Eq. "dequnt" subtracts it;
//       taken literally T_min would map to 2*T_min/s.  Used here:
//       zp = rint(m_min/s), code = rint(m/s) - zp, restore (code + zp) * s.
//   R2  one sign bit only: a b-bit level is 1 sign bit + a (b-1)-bit magnitude
//       code, Q_max(b) = 2^(b-1) - 1 (the formula and Algorithm 1 line 4 both
//       reserve the sign bit; it is reserved once).
//   R3  AIQ runs on magnitudes (Algorithm 1 line 2) with the per-token min/max
//       of the magnitudes; the sign is stored beside the code and applied after
//       dequantising.
//   R4  the algorithm is run independently per token row, n = H.
//   R5  zeroed outlier slots stay in the row (T_below keeps them): they take
//       part in min, max, delta and n, and receive code 0.
//   R6  returned level = the last level whose delta did not exceed Delta while
//       descending the candidate list from the top; the descent stops at the
//       first failure.  The top level is returned if the first lower one fails.
//   R7  candidates are an increasing list; the descent visits them in
//       decreasing order (a contiguous list reproduces Q <- Q-1).
//   R8  delta > Delta is evaluated exactly as  S > floor((double)Delta * H)
//       with S the integer numerator.
//   R9  rounding is to nearest, ties to even; T/s is the IEEE binary32 quotient.
//   R10 range == 0: s = m_max if m_max > 0 else 1.
//   R11 codes are clamped to [0, Q_max].
//   R12 NaN and +-Inf satisfy !(|x| < tau) and so travel as outliers.
//   R13 the sign plane carries the raw sign bit of inliers (so -0 round-trips);
//       outlier slots carry sign 0.
//   R14 scale is binary32, zero-point int32, CSR entries (column<<16 | raw16),
//       row pointers u32, columns ascending.
//   R15 the reconstruction is the binary32 product rounded once (RNE) to the
//       16-bit input type.
//
// Variant "signed values" (flag 1, an alternative reading of Sec. II-C.2): Eq. "Proposed" is applied to the
// signed inliers themselves, without Algorithm 1 lines 1-2 (no sign / magnitude split): the per-token min and
// max are those of the signed values of T_below (outlier slots count as +0), a b-bit level spends all b bits on
// the code, Q_max(b) = 2^b - 1, the zero-point rint(T_min / s) may be negative, and there is no sign plane
// (plane k = bit k of the code); a range T_max - T_min that overflows binary32 counts as the largest finite
// binary32.  Everything else (TS, descent, distortion test, placement, restore
// (code + zp) * s rounded once to the 16-bit type) is as above.  The blob header marks it in bits[7].
//
// Parity pins: see tests/test_oracle_*.py.  The paper prints no numeric example
// for TS, AIQ or TAB-Q, so the choice among readings R1-R6 is pinned only by the
// internal consistency of its equations ("parity unpinned" for that choice);
// everything downstream of the readings is pinned by hand-derived rows, closed
// forms, library cross-checks, error bounds and brute-force enumeration.

#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>

namespace {

constexpr uint32_t kMagic = 0x31515354u;  // bytes 'T','S','Q','1'
constexpr uint32_t kVersion = 1u;
constexpr int kF16 = 0;
constexpr int kBF16 = 1;

enum Status : int {
  kOk = 0,
  kInvalidArg = 1,
  kUnsupported = 2,
  kBufferTooSmall = 3,
  kCuda = 4,  // never produced here; keeps numbering aligned with the blob status field
  kCorruptBlob = 5,
  kOutlierOverflow = 6,
  kTimeout = 7
};

// ---- 16-bit <-> binary32, written from the IEEE 754 definitions -------------------

float bits_to_float(uint32_t u) {
  float f;
  std::memcpy(&f, &u, 4);
  return f;
}
uint32_t float_to_bits(float f) {
  uint32_t u;
  std::memcpy(&u, &f, 4);
  return u;
}

// binary16: 1 sign, 5 exponent (bias 15), 10 fraction.
float f16_to_float(uint16_t h) {
  const uint32_t sign = (uint32_t)(h >> 15) << 31;
  const int e = (h >> 10) & 0x1f;
  const uint32_t frac = h & 0x3ffu;
  if (e == 0x1f) return bits_to_float(sign | 0x7f800000u | (frac << 13));  // Inf / NaN
  if (e == 0) {
    // subnormal or zero: value = frac * 2^-24, exact in binary32
    float v = std::ldexp((float)frac, -24);
    return sign ? -v : v;
  }
  return bits_to_float(sign | ((uint32_t)(e - 15 + 127) << 23) | (frac << 13));
}

// bfloat16: the upper 16 bits of binary32.
float bf16_to_float(uint16_t h) { return bits_to_float((uint32_t)h << 16); }

// Round a non-negative finite-or-infinite binary32 to the nearest binary16, ties to even.
uint16_t float_to_f16_rne_nonneg(float f) {
  const uint32_t u = float_to_bits(f);
  const int e = (int)(u >> 23) & 0xff;
  const uint32_t frac = u & 0x7fffffu;
  if (e == 0xff) return frac ? 0x7e00 : 0x7c00;
  // value = sig * 2^(e-150) with sig = frac | 2^23 for normals, frac for subnormals
  const uint64_t sig = (e == 0) ? frac : (frac | 0x800000u);
  const int exp2 = (e == 0) ? -149 : e - 150;
  if (sig == 0) return 0;
  // target quantum: binary16 normal with unbiased exponent E has quantum 2^(E-10), E >= -14;
  // below that the quantum is fixed at 2^-24.
  int msb = 63 - __builtin_clzll(sig);
  int E = msb + exp2;  // floor(log2(value))
  int quantum = (E < -14) ? -24 : E - 10;
  int shift = quantum - exp2;  // number of low bits to drop (may be <= 0)
  uint64_t q;
  if (shift <= 0) {
    q = sig << (-shift);
  } else if (shift > 60) {
    q = 0;
  } else {
    const uint64_t rem = sig & ((1ull << shift) - 1);
    const uint64_t half = 1ull << (shift - 1);
    q = sig >> shift;
    if (rem > half || (rem == half && (q & 1))) q += 1;
  }
  // q counts quanta.  Re-normalise: a carry may push it to 2^11 (normal) or to 2^10 (subnormal -> normal).
  if (quantum == -24) {
    // subnormal range: q in [0, 1024]; 1024 is exactly the smallest normal (pattern 0x0400)
    return (uint16_t)q;
  }
  if (q == (1ull << 11)) {
    q >>= 1;
    E += 1;
  }
  if (E > 15) return 0x7c00;  // overflow to +Inf
  return (uint16_t)(((uint32_t)(E + 15) << 10) | ((uint32_t)q & 0x3ffu));
}

// Round a non-negative binary32 to the nearest bfloat16, ties to even.
uint16_t float_to_bf16_rne_nonneg(float f) {
  const uint32_t u = float_to_bits(f);
  if ((u & 0x7f800000u) == 0x7f800000u) {
    return (u & 0x7fffffu) ? 0x7fc0 : 0x7f80;
  }
  const uint32_t low = u & 0xffffu;
  uint32_t hi = u >> 16;
  if (low > 0x8000u || (low == 0x8000u && (hi & 1u))) hi += 1;  // carry may reach Inf: correct
  return (uint16_t)hi;
}

uint16_t float_to_raw16_nonneg(int dtype, float f);
// signed binary32 -> 16-bit pattern, round to nearest even on the magnitude, sign kept
uint16_t float_to_raw16_signed(int dtype, float f) {
  const uint32_t u = float_to_bits(f);
  const uint16_t mag = float_to_raw16_nonneg(dtype, bits_to_float(u & 0x7fffffffu));
  return (uint16_t)(mag | ((u >> 31) << 15));
}

float raw16_to_float(int dtype, uint16_t r) {
  return dtype == kF16 ? f16_to_float(r) : bf16_to_float(r);
}
uint16_t float_to_raw16_nonneg(int dtype, float f) {
  return dtype == kF16 ? float_to_f16_rne_nonneg(f) : float_to_bf16_rne_nonneg(f);
}

// ---- blob layout ---------------------------------------------------------------------
// header (64 B) | bits[T] u8 | scale[T] f32 | zp[T] i32 | word_off[T+1] u32 |
// out_ptr[T+1] u32 | words[T*bmax*WPP] u32 | outl[capacity] u32 ; every section starts
// on a 16-byte boundary.  Inside a token's b*WPP words the planes are interleaved per group of
// 32 elements: word g*b + k is plane k of elements 32g .. 32g+31.

struct Header {
  uint32_t magic, version, dtype, hidden, tokens, n_bits;
  uint8_t bits[8];
  float tau, delta;
  uint64_t total_words, total_outliers;
  uint32_t status, outlier_capacity;
};
static_assert(sizeof(Header) == 64, "header is 64 bytes");

struct Layout {
  uint64_t off_bits, off_scale, off_zp, off_word_off, off_out_ptr, off_words, off_outl, total;
  uint64_t wpp, words_capacity, outlier_capacity;
};

uint64_t align16(uint64_t v) { return (v + 15u) & ~(uint64_t)15u; }

bool make_layout(int64_t hidden, int64_t tokens, int bmax, int64_t max_outliers, Layout* L) {
  if (hidden < 1 || hidden > 65536 || tokens < 0 || bmax < 2 || bmax > 8) return false;
  const uint64_t T = (uint64_t)tokens, H = (uint64_t)hidden;
  if (T * H >= (1ull << 32)) return false;
  L->wpp = (H + 31) / 32;
  L->words_capacity = T * (uint64_t)bmax * L->wpp;
  if (L->words_capacity >= (1ull << 32)) return false;
  uint64_t cap = T * H;
  if (max_outliers > 0 && (uint64_t)max_outliers < cap) cap = (uint64_t)max_outliers;
  L->outlier_capacity = cap;
  uint64_t o = 64;
  L->off_bits = o;      o = align16(o + T);
  L->off_scale = o;     o = align16(o + 4 * T);
  L->off_zp = o;        o = align16(o + 4 * T);
  L->off_word_off = o;  o = align16(o + 4 * (T + 1));
  L->off_out_ptr = o;   o = align16(o + 4 * (T + 1));
  L->off_words = o;     o = align16(o + 4 * L->words_capacity);
  L->off_outl = o;      o = align16(o + 4 * cap);
  L->total = o;
  return true;
}

bool check_bits(const int32_t* bits, int n_bits) {
  if (!bits || n_bits < 1 || n_bits > 7) return false;
  for (int i = 0; i < n_bits; ++i) {
    if (bits[i] < 2 || bits[i] > 8) return false;
    if (i && bits[i] <= bits[i - 1]) return false;
  }
  return true;
}

// ---- TS: Eq. "ts" -------------------------------------------------------------------------
// Fills m[j] (magnitude of T_below, +0 in outlier slots), sg[j] (raw sign bit of inliers),
// is_out[j]; returns the number of outliers.
int64_t threshold_split(int dtype, const uint16_t* row, int64_t H, float tau, float* m, uint8_t* sg,
                        uint8_t* is_out) {
  int64_t n_out = 0;
  for (int64_t j = 0; j < H; ++j) {
    const float v = raw16_to_float(dtype, row[j]);
    const float a = std::fabs(v);
    const bool out = !(a < tau);  // |T_ij| >= tau; NaN lands here too (R12)
    is_out[j] = out ? 1 : 0;
    if (out) {
      m[j] = 0.0f;
      sg[j] = 0;
      ++n_out;
    } else {
      m[j] = a;
      sg[j] = (uint8_t)(row[j] >> 15);
    }
  }
  return n_out;
}

// ---- AIQ: Eq. "Proposed", on the magnitudes of one row, at level b --------------------------
void aiq(const float* m, int64_t H, float mmin, float mmax, int b, float* s_out, int32_t* zp_out,
         int32_t* q) {
  const int32_t qmax = (1 << (b - 1)) - 1;
  const float range = mmax - mmin;
  float s;
  if (range > 0.0f) {
    s = range / (float)qmax;
  } else {
    s = (mmax > 0.0f) ? mmax : 1.0f;  // R10
  }
  const int32_t zp = (int32_t)std::rint(mmin / s);
  for (int64_t j = 0; j < H; ++j) {
    int32_t c = (int32_t)std::rint(m[j] / s) - zp;
    if (c < 0) c = 0;
    if (c > qmax) c = qmax;
    q[j] = c;
  }
  *s_out = s;
  *zp_out = zp;
}

// ---- variant "signed values": AIQ on the signed inliers, Q_max = 2^b - 1 ---------------------------------
// v[j] = the signed value of T_below (outlier slots +0).
void signed_values(int dtype, const uint16_t* row, int64_t H, const uint8_t* is_out, float* v) {
  for (int64_t j = 0; j < H; ++j) v[j] = is_out[j] ? 0.0f : raw16_to_float(dtype, row[j]);
}

void aiq_signed(const float* v, int64_t H, float vmin, float vmax, int b, float* s_out, int32_t* zp_out, int32_t* q) {
  const int32_t qmax = (1 << b) - 1;
  float range = vmax - vmin;
  // Two finite values of opposite sign can lie further apart than binary32 holds (bf16 rows spanning more than
  // 3.4e38): the difference then counts as the largest finite binary32, so that scale and codes stay finite.
  if (range > 3.40282346638528859811704183484516925e+38f) range = 3.40282346638528859811704183484516925e+38f;
  float s;
  if (range > 0.0f) {
    s = range / (float)qmax;
  } else {
    const float c = std::fabs(vmax);  // a constant row: one level at the value itself (R10 carried over)
    s = (c > 0.0f) ? c : 1.0f;
  }
  const int32_t zp = (int32_t)std::rint(vmin / s);
  for (int64_t j = 0; j < H; ++j) {
    int32_t c = (int32_t)std::rint(v[j] / s) - zp;
    if (c < 0) c = 0;
    if (c > qmax) c = qmax;
    q[j] = c;
  }
  *s_out = s;
  *zp_out = zp;
}

void row_min_max(const float* m, int64_t H, float* mmin, float* mmax) {
  float lo = m[0], hi = m[0];
  for (int64_t j = 1; j < H; ++j) {
    if (m[j] < lo) lo = m[j];
    if (m[j] > hi) hi = m[j];
  }
  *mmin = lo;
  *mmax = hi;
}

// Numerator of delta in Algorithm 1 line 9 for a lower level b against the top level's codes q0.
int64_t distortion_sum(const int32_t* q0, const int32_t* q, int64_t H, int bmax, int b) {
  int64_t S = 0;
  for (int64_t j = 0; j < H; ++j) {
    const int32_t a = q0[j] >> (bmax - b);  // floor(T0 / 2^(Qbar - Q)), codes are non-negative
    const int32_t d = a - q[j];
    S += d < 0 ? -d : d;
  }
  return S;
}

int64_t s_max_of(float delta, int64_t H) { return (int64_t)std::floor((double)delta * (double)H); }

// ---- TAB-Q on one row: Algorithm 1 with reading R6 -----------------------------------------
struct RowResult {
  int b;
  float s;
  int32_t zp;
};

RowResult tabq_row(const float* m, int64_t H, const int32_t* bits, int n_bits, int64_t s_max,
                   std::vector<int32_t>& q0, std::vector<int32_t>& q, std::vector<int32_t>& qbest, bool signed_values_variant = false) {
  float mmin, mmax;
  row_min_max(m, H, &mmin, &mmax);
  const int bmax = bits[n_bits - 1];
  RowResult best;
  best.b = bmax;
  const auto quantise = [&](int b, float* s, int32_t* zp, int32_t* out) {
    if (signed_values_variant) {
      aiq_signed(m, H, mmin, mmax, b, s, zp, out);
    } else {
      aiq(m, H, mmin, mmax, b, s, zp, out);
    }
  };
  quantise(bmax, &best.s, &best.zp, q0.data());
  qbest = q0;
  for (int i = n_bits - 2; i >= 0; --i) {
    const int b = bits[i];
    float s;
    int32_t zp;
    quantise(b, &s, &zp, q.data());
    const int64_t S = distortion_sum(q0.data(), q.data(), H, bmax, b);
    if (S > s_max) break;  // delta > Delta: stop, keep the last passing level
    best.b = b;
    best.s = s;
    best.zp = zp;
    qbest = q;
  }
  return best;
}

}  // namespace

extern "C" {

// Section offsets and total size of a blob for `tokens` rows. offsets[0..6] = bits, scale, zp,
// word_off, out_ptr, words, outl; offsets[7] = total bytes; offsets[8] = outlier capacity.
int tsq_ref_layout(int hidden, long long tokens, int bmax, long long max_outliers,
                   unsigned long long* offsets) {
  Layout L;
  if (!offsets || !make_layout(hidden, tokens, bmax, max_outliers, &L)) return kInvalidArg;
  offsets[0] = L.off_bits;
  offsets[1] = L.off_scale;
  offsets[2] = L.off_zp;
  offsets[3] = L.off_word_off;
  offsets[4] = L.off_out_ptr;
  offsets[5] = L.off_words;
  offsets[6] = L.off_outl;
  offsets[7] = L.total;
  offsets[8] = L.outlier_capacity;
  return kOk;
}

// Encode x[tokens][hidden] (raw 16-bit patterns, host memory) into blob (host memory).
// The whole blob is zero-filled first, so unused capacity reads as zero.
int tsq_ref_encode_ex(int dtype, int hidden, long long tokens, float tau, const int32_t* bits,
                      int n_bits, float delta, long long max_outliers, int flags, const uint16_t* x,
                      uint8_t* blob, unsigned long long blob_bytes) {
  if ((dtype != kF16 && dtype != kBF16) || !check_bits(bits, n_bits) || !blob) return kInvalidArg;
  if (flags != 0 && flags != 1) return kInvalidArg;
  const bool sv = flags == 1;  // variant "signed values"
  if (tau != tau || delta != delta) return kInvalidArg;
  if (tokens > 0 && !x) return kInvalidArg;
  const int bmax = bits[n_bits - 1];
  Layout L;
  if (!make_layout(hidden, tokens, bmax, max_outliers, &L)) return kInvalidArg;
  if (blob_bytes < L.total) return kBufferTooSmall;
  std::memset(blob, 0, L.total);

  const int64_t H = hidden, T = tokens;
  const int64_t s_max = s_max_of(delta, H);
  uint8_t* o_bits = blob + L.off_bits;
  float* o_scale = reinterpret_cast<float*>(blob + L.off_scale);
  int32_t* o_zp = reinterpret_cast<int32_t*>(blob + L.off_zp);
  uint32_t* o_word_off = reinterpret_cast<uint32_t*>(blob + L.off_word_off);
  uint32_t* o_out_ptr = reinterpret_cast<uint32_t*>(blob + L.off_out_ptr);
  uint32_t* o_words = reinterpret_cast<uint32_t*>(blob + L.off_words);
  uint32_t* o_outl = reinterpret_cast<uint32_t*>(blob + L.off_outl);

  std::vector<float> m(H);
  std::vector<uint8_t> sg(H), is_out(H);
  std::vector<int32_t> q0(H), q(H), qbest(H);
  uint64_t word_off = 0, out_ptr = 0;
  uint32_t status = kOk;
  o_word_off[0] = 0;
  o_out_ptr[0] = 0;
  for (int64_t t = 0; t < T; ++t) {
    const uint16_t* row = x + t * H;
    threshold_split(dtype, row, H, tau, m.data(), sg.data(), is_out.data());
    // CSR row of T_above: ascending columns, original 16-bit patterns.
    for (int64_t j = 0; j < H; ++j) {
      if (!is_out[j]) continue;
      if (out_ptr < L.outlier_capacity) {
        o_outl[out_ptr] = ((uint32_t)j << 16) | row[j];
      } else {
        status = kOutlierOverflow;  // entry dropped; counts keep running
      }
      ++out_ptr;
    }
    if (sv) signed_values(dtype, row, H, is_out.data(), m.data());  // m now holds the signed values of T_below
    const RowResult r = tabq_row(m.data(), H, bits, n_bits, s_max, q0, q, qbest, sv);
    o_bits[t] = (uint8_t)r.b;
    o_scale[t] = r.s;
    o_zp[t] = r.zp;
    // bit-planes: plane 0 = sign, plane 1+k = bit k of the magnitude code.  Group g holds
    // elements 32g .. 32g+31 and owns words g*b .. g*b + b-1 (one word per plane); bit i of a
    // group's word belongs to element 32g + i; pad bits stay 0.
    uint32_t* wrow = o_words + word_off;
    for (int64_t j = 0; j < H; ++j) {
      const uint64_t g = (uint64_t)j >> 5;
      const uint32_t bit = 1u << (j & 31);
      if (sv) {  // no sign plane: plane k = bit k of the b-bit code
        for (int k = 0; k < r.b; ++k) {
          if ((qbest[j] >> k) & 1) wrow[g * r.b + k] |= bit;
        }
        continue;
      }
      if (sg[j]) wrow[g * r.b] |= bit;
      for (int k = 0; k < r.b - 1; ++k) {
        if ((qbest[j] >> k) & 1) wrow[g * r.b + 1 + k] |= bit;
      }
    }
    word_off += (uint64_t)r.b * L.wpp;
    o_word_off[t + 1] = (uint32_t)word_off;
    o_out_ptr[t + 1] = (uint32_t)out_ptr;
  }

  Header h;
  std::memset(&h, 0, sizeof h);
  h.magic = kMagic;
  h.version = kVersion;
  h.dtype = (uint32_t)dtype;
  h.hidden = (uint32_t)hidden;
  h.tokens = (uint32_t)tokens;
  h.n_bits = (uint32_t)n_bits;
  for (int i = 0; i < n_bits; ++i) h.bits[i] = (uint8_t)bits[i];
  h.bits[7] = (uint8_t)flags;  // n_bits <= 7: the last entry is free and carries the variant
  h.tau = tau;
  h.delta = delta;
  h.total_words = word_off;
  h.total_outliers = out_ptr;
  h.status = status;
  h.outlier_capacity = (uint32_t)L.outlier_capacity;
  std::memcpy(blob, &h, sizeof h);
  return kOk;
}

int tsq_ref_encode(int dtype, int hidden, long long tokens, float tau, const int32_t* bits,
                   int n_bits, float delta, long long max_outliers, const uint16_t* x,
                   uint8_t* blob, unsigned long long blob_bytes) {
  return tsq_ref_encode_ex(dtype, hidden, tokens, tau, bits, n_bits, delta, max_outliers, 0, x, blob, blob_bytes);
}

// Variant "signed values": AIQ at level b on a row of binary32 signed values (already threshold-split).
int tsq_ref_aiq_signed(const float* v, int hidden, int b, float* s, int32_t* zp, int32_t* q) {
  if (!v || hidden < 1 || b < 2 || b > 8 || !s || !zp || !q) return kInvalidArg;
  float vmin, vmax;
  row_min_max(v, hidden, &vmin, &vmax);
  aiq_signed(v, hidden, vmin, vmax, b, s, zp, q);
  return kOk;
}

// Decode a blob into y[tokens][hidden] (raw 16-bit patterns). Eq. "dequnt".
int tsq_ref_decode(const uint8_t* blob, unsigned long long blob_bytes, uint16_t* y) {
  if (!blob || blob_bytes < 64) return kInvalidArg;
  Header h;
  std::memcpy(&h, blob, sizeof h);
  if (h.magic != kMagic || h.version != kVersion) return kCorruptBlob;
  if (h.dtype != (uint32_t)kF16 && h.dtype != (uint32_t)kBF16) return kCorruptBlob;
  if (h.n_bits < 1 || h.n_bits > 7) return kCorruptBlob;
  if (h.status != kOk) return (int)h.status;
  if (h.bits[7] > 1) return kCorruptBlob;
  const bool sv = h.bits[7] == 1;
  const int bmax = h.bits[h.n_bits - 1];
  Layout L;
  if (!make_layout(h.hidden, h.tokens, bmax, h.outlier_capacity, &L)) return kCorruptBlob;
  if (h.tokens > 0 && L.outlier_capacity != h.outlier_capacity) return kCorruptBlob;
  if (blob_bytes < L.total) return kBufferTooSmall;
  if (h.total_words > L.words_capacity || h.total_outliers > L.outlier_capacity) return kCorruptBlob;
  if (h.tokens > 0 && !y) return kInvalidArg;

  const int64_t H = h.hidden, T = h.tokens;
  const int dtype = (int)h.dtype;
  const uint8_t* i_bits = blob + L.off_bits;
  const float* i_scale = reinterpret_cast<const float*>(blob + L.off_scale);
  const int32_t* i_zp = reinterpret_cast<const int32_t*>(blob + L.off_zp);
  const uint32_t* i_word_off = reinterpret_cast<const uint32_t*>(blob + L.off_word_off);
  const uint32_t* i_out_ptr = reinterpret_cast<const uint32_t*>(blob + L.off_out_ptr);
  const uint32_t* i_words = reinterpret_cast<const uint32_t*>(blob + L.off_words);
  const uint32_t* i_outl = reinterpret_cast<const uint32_t*>(blob + L.off_outl);

  for (int64_t t = 0; t < T; ++t) {
    const int b = i_bits[t];
    if (b < 2 || b > bmax) return kCorruptBlob;
    const uint64_t wo = i_word_off[t];
    if (wo + (uint64_t)b * L.wpp > h.total_words) return kCorruptBlob;
    if (i_word_off[t + 1] != wo + (uint64_t)b * L.wpp) return kCorruptBlob;
    const uint32_t p0 = i_out_ptr[t], p1 = i_out_ptr[t + 1];
    if (p1 < p0 || p1 > h.total_outliers) return kCorruptBlob;
    const float s = i_scale[t];
    const int32_t zp = i_zp[t];
    const uint32_t* wrow = i_words + wo;
    uint16_t* yrow = y + t * H;
    for (int64_t j = 0; j < H; ++j) {
      const uint64_t g = (uint64_t)j >> 5;
      const int sh = (int)(j & 31);
      if (sv) {
        int32_t q = 0;
        for (int k = 0; k < b; ++k) q |= (int32_t)((wrow[g * b + k] >> sh) & 1u) << k;
        yrow[j] = float_to_raw16_signed(dtype, (float)(q + zp) * s);  // signed product, rounded once
        continue;
      }
      int32_t q = 0;
      for (int k = 0; k < b - 1; ++k) q |= (int32_t)((wrow[g * b + 1 + k] >> sh) & 1u) << k;
      const uint32_t sign = (wrow[g * b] >> sh) & 1u;
      const float mag = (float)(q + zp) * s;              // (T^ - Z) .* S with Z = -zp (R1)
      const uint16_t hbits = float_to_raw16_nonneg(dtype, mag);  // R15
      yrow[j] = (uint16_t)(hbits | (sign << 15));
    }
    // "+ T_above": the slot decodes to +0, so adding the outlier equals overwriting it.
    for (uint32_t p = p0; p < p1; ++p) {
      const uint32_t e = i_outl[p];
      const uint32_t col = e >> 16;
      if ((int64_t)col >= H) return kCorruptBlob;
      yrow[col] = (uint16_t)(e & 0xffffu);
    }
  }
  return kOk;
}

// ---- introspection used by the pins -------------------------------------------------------

// TS on one row: magnitudes of T_below as binary32, sign bits, outlier flags.
int tsq_ref_ts_row(int dtype, const uint16_t* row, int hidden, float tau, float* m, uint8_t* sg,
                   uint8_t* is_out, long long* n_out) {
  if (!row || hidden < 1 || !m || !sg || !is_out) return kInvalidArg;
  const int64_t n = threshold_split(dtype, row, hidden, tau, m, sg, is_out);
  if (n_out) *n_out = n;
  return kOk;
}

// AIQ at level b on a row of binary32 magnitudes (already threshold-split).
int tsq_ref_aiq(const float* m, int hidden, int b, float* s, int32_t* zp, int32_t* q) {
  if (!m || hidden < 1 || b < 2 || b > 8 || !s || !zp || !q) return kInvalidArg;
  float mmin, mmax;
  row_min_max(m, hidden, &mmin, &mmax);
  aiq(m, hidden, mmin, mmax, b, s, zp, q);
  return kOk;
}

// Distortion numerators S_b for every candidate below the top one (S[n_bits-1] = 0), and the
// level Algorithm 1 returns for tolerance delta.
int tsq_ref_select(const float* m, int hidden, const int32_t* bits, int n_bits, float delta,
                   long long* S, int* b_star) {
  if (!m || hidden < 1 || !check_bits(bits, n_bits)) return kInvalidArg;
  const int64_t H = hidden;
  float mmin, mmax;
  row_min_max(m, H, &mmin, &mmax);
  const int bmax = bits[n_bits - 1];
  std::vector<int32_t> q0(H), q(H), qbest(H);
  float s;
  int32_t zp;
  aiq(m, H, mmin, mmax, bmax, &s, &zp, q0.data());
  if (S) {
    S[n_bits - 1] = 0;
    for (int i = 0; i < n_bits - 1; ++i) {
      aiq(m, H, mmin, mmax, bits[i], &s, &zp, q.data());
      S[i] = distortion_sum(q0.data(), q.data(), H, bmax, bits[i]);
    }
  }
  if (b_star) {
    const RowResult r = tabq_row(m, H, bits, n_bits, s_max_of(delta, H), q0, q, qbest);
    *b_star = r.b;
  }
  return kOk;
}

// 16-bit conversions, exposed so the pins can compare them with a library's.
float tsq_ref_raw16_to_float(int dtype, uint16_t r) { return raw16_to_float(dtype, r); }
uint16_t tsq_ref_float_to_raw16(int dtype, float f) {
  const uint32_t u = float_to_bits(f);
  const uint16_t mag = float_to_raw16_nonneg(dtype, bits_to_float(u & 0x7fffffffu));
  return (uint16_t)(mag | ((u >> 31) << 15));
}

}  // extern "C"
