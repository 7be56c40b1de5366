"""Size and latency models (Eq. "bkv", Eq. "if_total", epsilon-outage latency, rate search): the oracle against what
the paper's formulas fix, then the library's host functions (C ABI, no GPU needed) against the oracle."""
import math

import pytest

from oracle import model_ref as M
from paper_2511_04002_b200 import binding as B


# ------------------------------------------------------------------ oracle pins

def test_kv_bits_closed_form_for_one_bit_width():
    # all layers at Q bits: 2 Q HD (l w + (L - l)(w - 1)) + HD Q
    for (w, l, L, hd, q) in [(1, 1, 1, 8, 4.0), (50, 20, 32, 4096, 4.0), (7, 32, 32, 5120, 3.0), (128, 1, 40, 128, 16.0)]:
        want = 2 * q * hd * (l * w + (L - l) * (w - 1)) + hd * q
        assert M.kv_bits(w, l, L, L + 1, hd, q, 99.0) == want          # split beyond the last layer: front bits everywhere
        assert M.kv_bits(w, l, L, 1, hd, 99.0, q) == want              # split at layer 1: back bits everywhere


def test_kv_bits_hand_example_with_two_bit_widths():
    # w = 3, l = 2, L = 4, split at layer 3, HD = 10, Q_a1 = 4, Q_a2 = 8:
    # layers 1, 2 (front, 4 bits) hold T_3 = 30: 2 * (30*4 + 30*4) = 480; layers 3, 4 (back, 8 bits) hold T_2 = 20:
    # 2 * (20*8 + 20*8) = 640; hidden state of token 3 at layer 2 (front): 10 * 4 = 40
    assert M.kv_bits(3, 2, 4, 3, 10, 4.0, 8.0) == 480 + 640 + 40
    # exit at layer 3 instead: layers 1, 2 at 4 bits and layer 3 at 8 bits hold T_3, layer 4 holds T_2, hidden at 8 bits
    assert M.kv_bits(3, 3, 4, 3, 10, 4.0, 8.0) == 2 * (120 + 120 + 240) + 2 * 160 + 80


def test_kv_bits_grows_by_one_token_per_layer():
    # one more token adds 2 HD Q_k at every layer (Eq. "bkv" is linear in w)
    a, b = M.kv_bits(10, 5, 12, 7, 64, 4.0, 8.0), M.kv_bits(11, 5, 12, 7, 64, 4.0, 8.0)
    assert b - a == 2 * 64 * (6 * 4.0 + 6 * 8.0)


def test_io_bits_switch():
    assert M.io_bits(9, 4, 8, 5, 32, 4.0, 8.0, True) == M.kv_bits(9, 4, 8, 5, 32, 4.0, 8.0)
    assert M.io_bits(9, 4, 8, 5, 32, 4.0, 8.0, False) == 9 * 32 * 4.0
    assert M.io_bits(9, 6, 8, 5, 32, 4.0, 8.0, False) == 9 * 32 * 8.0     # layer 6 lies in the back segment


def test_outage_limits_and_inverse():
    W, snr = 10e6, 10.0
    assert M.outage(1e-3, W, snr) < 1e-10                                  # R -> 0: no outage
    assert M.outage(50 * W, W, snr) == 1.0                                  # R >> W log2(1 + snr): certain outage
    # P_o(R) = p  <=>  R = W log2(1 - gamma ln(1 - p))
    for p in (0.001, 0.1, 0.5, 0.9):
        R = W * math.log2(1.0 - snr * math.log(1.0 - p))
        assert abs(M.outage(R, W, snr) - p) < 1e-12
    assert M.outage(2e7, W, snr) < M.outage(3e7, W, snr)                    # increasing in R


def test_latency_counts_retransmissions():
    W, snr = 10e6, 10.0
    R = W * math.log2(1.0 - snr * math.log(1.0 - 0.1))                      # P_o = 0.1
    assert M.latency(1e6, R, W, snr, 0.1 * 1.0000001) == 1e6 / R * 1        # eps just above P_o: one transmission is enough
    assert M.latency(1e6, R, W, snr, 0.001 * 1.0000001) == 1e6 / R * 3      # 0.1^3 = 0.001
    assert M.latency(1e6, R, W, snr, 0.001 * 0.99) == 1e6 / R * 4
    assert M.latency(2e6, R, W, snr, 0.01) == 2 * M.latency(1e6, R, W, snr, 0.01)


def test_best_rate_is_the_grid_minimum_and_respects_the_interval():
    W, snr = 10e6, 10.0
    lo, hi = 1e6, 80e6
    r = M.best_rate(lo, hi, W, snr, points=20001)
    for probe in (lo, hi, 0.5 * r, 0.9 * r, min(hi, 1.1 * r)):
        assert M.g(r, W, snr) <= M.g(probe, W, snr) + 1e-18
    assert M.best_rate(2e6, 2e6, W, snr, points=3) == 2e6


# ------------------------------------------------------------------ the library's host functions against the oracle

CASES = [(1, 1, 1, 1, 8, 4.0, 4.0), (50, 20, 32, 20, 4096, 4.0, 16.0), (50, 20, 40, 20, 5120, 3.0, 16.0),
         (2048, 32, 32, 21, 4096, 4.0, 8.0), (7, 1, 80, 40, 8192, 2.0, 16.0), (3, 2, 4, 3, 10, 4.0, 8.0)]


@pytest.mark.parametrize("case", CASES)
def test_library_sizes_equal_the_oracle(case):
    w, l, L, split, hd, q1, q2 = case
    assert B.model_kv_bits(w, l, L, split, hd, q1, q2) == M.kv_bits(w, l, L, split, hd, q1, q2)
    for send in (True, False):
        assert B.model_io_bits(w, l, L, split, hd, q1, q2, send) == M.io_bits(w, l, L, split, hd, q1, q2, send)


def test_library_link_model_equals_the_oracle():
    W, snr = 10e6, 10.0                                   # the paper's link: 10 MHz, gamma = 10, epsilon = 0.001
    for R in (1e5, 1e6, 5e6, 2e7, 3.3e7, 6e7):
        assert math.isclose(B.model_outage(R, W, snr), M.outage(R, W, snr), rel_tol=1e-13, abs_tol=1e-300)
        for eps in (0.001, 0.05):
            assert math.isclose(B.model_latency(3.5e6, R, W, snr, eps), M.latency(3.5e6, R, W, snr, eps), rel_tol=1e-12)
    for (lo, hi) in [(1e6, 80e6), (1e6, 5e6), (3e7, 4e7)]:
        r_lib, r_ref = B.model_best_rate(lo, hi, W, snr), M.best_rate(lo, hi, W, snr)
        assert abs(r_lib - r_ref) <= (hi - lo) / 1e5 + 1e-9 * hi          # the oracle's grid step
        assert M.g(r_lib, W, snr) <= M.g(r_ref, W, snr) * (1 + 1e-9)


def test_library_rejects_arguments_outside_the_ranges():
    assert math.isnan(B.model_kv_bits(0, 1, 4, 2, 8, 4.0, 8.0))
    assert math.isnan(B.model_kv_bits(3, 5, 4, 2, 8, 4.0, 8.0))
    assert math.isnan(B.model_io_bits(3, 1, 4, 2, 0, 4.0, 8.0, True))
    assert math.isnan(B.model_outage(0.0, 1e7, 10.0))
    assert math.isnan(B.model_latency(1e6, 1e6, 1e7, 10.0, 1.5))
    assert math.isnan(B.model_best_rate(5e6, 1e6, 1e7, 10.0))
