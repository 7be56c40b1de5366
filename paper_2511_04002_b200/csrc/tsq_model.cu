// Host-side size and latency models around the codec (Sec. II-B: Eq. "bkv", Eq. "if_total"; Sec. II-D.2: the
// epsilon-outage latency and the rate search), so that a caller can take the early-exit decisions of
// Algorithm 2 ("compress harder", "drop the KV cache") from the payload sizes tsq_blob_info reports.
// Plain double arithmetic, no device work, no state.

#include <cmath>
#include <limits>

#include "tsq.h"

namespace {

const double kNaN = std::numeric_limits<double>::quiet_NaN();

bool layers_ok(int64_t w, int32_t layer, int32_t n_layers, int32_t split_layer, int64_t hd, double qa_front, double qa_back) {
  return w >= 1 && n_layers >= 1 && layer >= 1 && layer <= n_layers && split_layer >= 1 && hd >= 1 && qa_front >= 0.0 &&
         qa_back >= 0.0;
}

// activation bit-width of layer k: the front segment's below the split layer, the back segment's from it on
double qa_of(int32_t k, int32_t split_layer, double qa_front, double qa_back) { return k < split_layer ? qa_front : qa_back; }

double outage(double rate, double bandwidth, double snr) {
  return 1.0 - std::exp(-(std::exp2(rate / bandwidth) - 1.0) / snr);
}

double g_of(double rate, double bandwidth, double snr) { return std::log(1.0 / outage(rate, bandwidth, snr)) / rate; }

}  // namespace

extern "C" {

double tsq_model_kv_bits(int64_t w, int32_t layer, int32_t n_layers, int32_t split_layer, int64_t hd, double qa_front,
                         double qa_back) {
  if (!layers_ok(w, layer, n_layers, split_layer, hd, qa_front, qa_back)) return kNaN;
  const double t_w = static_cast<double>(w) * static_cast<double>(hd);        // T_w: elements of K (or V) for w tokens
  const double t_prev = static_cast<double>(w - 1) * static_cast<double>(hd);  // T_{w-1}
  double bits = 0.0;
  for (int32_t k = 1; k <= layer; ++k) bits += 2.0 * t_w * qa_of(k, split_layer, qa_front, qa_back);
  for (int32_t k = layer + 1; k <= n_layers; ++k) bits += 2.0 * t_prev * qa_of(k, split_layer, qa_front, qa_back);
  return bits + static_cast<double>(hd) * qa_of(layer, split_layer, qa_front, qa_back);
}

double tsq_model_io_bits(int64_t w, int32_t layer, int32_t n_layers, int32_t split_layer, int64_t hd, double qa_front,
                         double qa_back, int32_t send_kv) {
  if (!layers_ok(w, layer, n_layers, split_layer, hd, qa_front, qa_back)) return kNaN;
  if (send_kv != 0) return tsq_model_kv_bits(w, layer, n_layers, split_layer, hd, qa_front, qa_back);
  return static_cast<double>(w) * static_cast<double>(hd) * qa_of(layer, split_layer, qa_front, qa_back);
}

double tsq_model_outage(double rate, double bandwidth, double snr) {
  if (!(rate > 0.0) || !(bandwidth > 0.0) || !(snr > 0.0)) return kNaN;
  return outage(rate, bandwidth, snr);
}

double tsq_model_latency(double bits, double rate, double bandwidth, double snr, double epsilon) {
  if (!(bits >= 0.0) || !(rate > 0.0) || !(bandwidth > 0.0) || !(snr > 0.0) || !(epsilon > 0.0) || !(epsilon < 1.0)) return kNaN;
  const double po = outage(rate, bandwidth, snr);
  if (!(po > 0.0)) return bits / rate;  // no outage at all: one transmission
  if (!(po < 1.0)) return std::numeric_limits<double>::infinity();
  return bits / rate * std::ceil(std::log(epsilon) / std::log(po));
}

double tsq_model_best_rate(double rate_lo, double rate_hi, double bandwidth, double snr) {
  if (!(rate_lo > 0.0) || !(rate_hi >= rate_lo) || !(bandwidth > 0.0) || !(snr > 0.0)) return kNaN;
  // one-dimensional search: a coarse scan for the best cell, then golden-section refinement inside its neighbourhood
  const int cells = 4096;
  int best = 0;
  double best_g = g_of(rate_lo, bandwidth, snr);
  for (int i = 1; i <= cells; ++i) {
    const double r = rate_lo + (rate_hi - rate_lo) * i / cells;
    const double g = g_of(r, bandwidth, snr);
    if (g < best_g) {
      best_g = g;
      best = i;
    }
  }
  double a = rate_lo + (rate_hi - rate_lo) * (best > 0 ? best - 1 : 0) / cells;
  double b = rate_lo + (rate_hi - rate_lo) * (best < cells ? best + 1 : cells) / cells;
  const double phi = 0.6180339887498949;
  double c = b - phi * (b - a), d = a + phi * (b - a);
  double gc = g_of(c, bandwidth, snr), gd = g_of(d, bandwidth, snr);
  for (int it = 0; it < 80 && b - a > 1e-12 * (1.0 + std::fabs(b)); ++it) {
    if (gc < gd) {
      b = d; d = c; gd = gc;
      c = b - phi * (b - a); gc = g_of(c, bandwidth, snr);
    } else {
      a = c; c = d; gc = gd;
      d = a + phi * (b - a); gd = g_of(d, bandwidth, snr);
    }
  }
  const double mid = 0.5 * (a + b);
  // an end of the interval wins when the function is monotone there
  double r = mid, g = g_of(mid, bandwidth, snr);
  if (g_of(rate_lo, bandwidth, snr) < g) { r = rate_lo; g = g_of(rate_lo, bandwidth, snr); }
  if (g_of(rate_hi, bandwidth, snr) < g) r = rate_hi;
  return r;
}

}  // extern "C"
