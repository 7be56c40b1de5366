"""CPU oracle of the size and latency models around the codec.

Test infrastructure only: a plain restatement of the paper's closed forms (Sec. II-B, Eq. "bkv" and
Eq. "if_total"; Sec. II-D.2, the epsilon-outage latency, P_o(R) and the rate search R* = argmin g(R)) in
Python floats (binary64), one term at a time, no shortcuts.  It shares nothing with the library's C code.
Pins: tests/test_model_pins.py (closed forms for equal bit-widths, limits, hand-computed values, brute force).
"""
from __future__ import annotations

import math


def qa_of(k: int, split_layer: int, qa_front: float, qa_back: float) -> float:
    """Activation bits of layer k: Q_a1 below the split layer, Q_a2 from it on (the case distinction under Eq. "bkv")."""
    return qa_front if k < split_layer else qa_back


def kv_bits(w: int, layer: int, n_layers: int, split_layer: int, hd: int, qa_front: float, qa_back: float) -> float:
    """Eq. "bkv": 2 sum_{k=1}^{l} T_w Q_k + 2 sum_{k=l+1}^{L} T_{w-1} Q_k + HD Q_l, with T_w = w HD."""
    t_w, t_prev = w * hd, (w - 1) * hd
    total = 0.0
    for k in range(1, layer + 1):
        total += 2 * t_w * qa_of(k, split_layer, qa_front, qa_back)
    for k in range(layer + 1, n_layers + 1):
        total += 2 * t_prev * qa_of(k, split_layer, qa_front, qa_back)
    return total + hd * qa_of(layer, split_layer, qa_front, qa_back)


def io_bits(w: int, layer: int, n_layers: int, split_layer: int, hd: int, qa_front: float, qa_back: float, send_kv: bool) -> float:
    """Eq. "if_total": I_kv B_kv + (1 - I_kv) T_w Q_l."""
    i_kv = 1 if send_kv else 0
    return i_kv * kv_bits(w, layer, n_layers, split_layer, hd, qa_front, qa_back) + \
        (1 - i_kv) * (w * hd) * qa_of(layer, split_layer, qa_front, qa_back)


def outage(rate: float, bandwidth: float, snr: float) -> float:
    """P_o(R) = 1 - exp(-(2^(R/W) - 1) / gamma)."""
    return 1.0 - math.exp(-(2.0 ** (rate / bandwidth) - 1.0) / snr)


def latency(bits: float, rate: float, bandwidth: float, snr: float, epsilon: float) -> float:
    """L_eps(D; R) = D / R * ceil(ln(eps) / ln(P_o(R)))."""
    po = outage(rate, bandwidth, snr)
    return bits / rate * math.ceil(math.log(epsilon) / math.log(po))


def g(rate: float, bandwidth: float, snr: float) -> float:
    return math.log(1.0 / outage(rate, bandwidth, snr)) / rate


def best_rate(rate_lo: float, rate_hi: float, bandwidth: float, snr: float, points: int = 200001) -> float:
    """R* = argmin_{R in [lo, hi]} g(R), by brute force over a dense grid."""
    best, best_g = rate_lo, g(rate_lo, bandwidth, snr)
    for i in range(1, points):
        r = rate_lo + (rate_hi - rate_lo) * i / (points - 1)
        v = g(r, bandwidth, snr)
        if v < best_g:
            best, best_g = r, v
    return best
