"""Pins for the oracle's "signed values" variant (AIQ on the signed inliers, no sign plane, Q_max = 2^b - 1).

No GPU, no CUDA path.  The variant is tied to: rows worked by hand, its reduction to the pinned magnitude
variant one level up on non-negative rows, the affine round-to-nearest closed form away from ties, the
s/2 error bound, an independent reader of the planes, and brute-force level selection on tiny rows.
"""
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import tsq_ref as R
from tests.test_oracle_pins import f16_raw, f32_to_raw, raw_to_f32

INF = float("inf")


def codes_of_planes(words_row, b, hidden):
    """Independent scalar reader: group g owns words g*b .. g*b+b-1, plane k = bit k of the code."""
    code = np.zeros(hidden, np.int64)
    for j in range(hidden):
        g, i = divmod(j, 32)
        for k in range(b):
            code[j] |= ((int(words_row[g * b + k]) >> i) & 1) << k
    return code


# ---------------------------------------------------------------- rows worked by hand

def test_hand_row_exact_grid():
    # range 3 over Q_max(2) = 3: s = 1, zp = rint(-1 / 1) = -1, codes v - (-1); the grid holds every value
    raw = f16_raw([[-1.0, 0.0, 1.0, 2.0]])
    blob = R.encode(raw, R.F16, INF, [2], signed_values=True)
    hdr, sec = R.header(blob), R.sections(blob)
    assert hdr["variant"] == 1 and hdr["bits"][:1] == [2] and hdr["total_words"] == 2
    assert (float(sec["scale"][0]), int(sec["zp"][0]), int(sec["bits"][0])) == (1.0, -1, 2)
    # codes 0,1,2,3: bit 0 set for elements 1 and 3, bit 1 for elements 2 and 3
    assert sec["words"].tolist() == [0b1010, 0b1100]
    assert np.array_equal(R.decode(blob), raw)


def test_hand_row_ties_and_clamp():
    # range 6 over 3: s = 2.  v/s = -1.5, -0.5, 0.5, 1.5 are all ties: rint -> -2, -0, 0, 2 (to even);
    # zp = -2; codes 0, 2, 2, 4 -> the last is clamped to 3; restored (code - 2) * 2 = -4, 0, 0, 2
    raw = f16_raw([[-3.0, -1.0, 1.0, 3.0]])
    blob = R.encode(raw, R.F16, INF, [2], signed_values=True)
    sec = R.sections(blob)
    assert (float(sec["scale"][0]), int(sec["zp"][0])) == (2.0, -2)
    assert codes_of_planes(sec["words"], 2, 4).tolist() == [0, 2, 2, 3]
    assert raw_to_f32(R.decode(blob)[0], R.F16).tolist() == [-4.0, 0.0, 0.0, 2.0]


def test_hand_row_with_outlier_slot_counting_as_zero():
    # 50 is an outlier (tau 10): its slot is +0 for min/max and coding, its value comes back from the CSR list.
    # inliers -6, +0(slot), 3, 9: range 15 over Q_max(4) = 15: s = 1, zp = -6, codes 0, 6, 9, 15
    raw = f16_raw([[-6.0, 50.0, 3.0, 9.0]])
    blob = R.encode(raw, R.F16, 10.0, [4], signed_values=True)
    sec = R.sections(blob)
    assert (float(sec["scale"][0]), int(sec["zp"][0])) == (1.0, -6)
    assert codes_of_planes(sec["words"], 4, 4).tolist() == [0, 6, 9, 15]
    assert sec["out_ptr"].tolist() == [0, 1] and int(sec["outl"][0]) == (1 << 16) | int(raw[0, 1])
    assert np.array_equal(R.decode(blob), raw)


def test_constant_rows():
    s, zp, q = R.aiq_signed(np.full(5, -2.5, np.float32), 3)
    assert (s, zp, q.tolist()) == (2.5, -1, [0] * 5)          # restore (0 - 1) * 2.5 = -2.5 exactly
    s, zp, q = R.aiq_signed(np.zeros(7, np.float32), 2)
    assert (s, zp, q.tolist()) == (1.0, 0, [0] * 7)
    raw = f16_raw([[-2.5] * 5])
    assert np.array_equal(R.decode(R.encode(raw, R.F16, INF, [3, 8], signed_values=True)), raw)


def test_range_beyond_binary32_counts_as_the_largest_finite_value():
    v = raw_to_f32(f32_to_raw(np.array([-3.0e38, 3.0e38, 0.0], np.float32), R.BF16), R.BF16)
    fmax = np.finfo(np.float32).max
    s, zp, q = R.aiq_signed(v, 2)
    assert np.float32(s) == np.float32(fmax) / np.float32(3)
    assert zp == int(np.rint(np.float32(v[0]) / np.float32(s))) == -3
    assert q.tolist() == [0, 3, 3]                               # rint(2.6) + 3 = 6 is clamped; 0 + 3 = 3
    y = R.decode(R.encode(f32_to_raw(v, R.BF16).reshape(1, 3), R.BF16, INF, [2], signed_values=True))
    assert np.all(~np.isnan(raw_to_f32(y[0], R.BF16)))


# ---------------------------------------------------------------- reduction to the magnitude variant

@pytest.mark.parametrize("b", [2, 3, 4, 7])
def test_non_negative_rows_equal_the_magnitude_variant_one_level_up(b):
    """With every value >= 0 the sign plane of the magnitude variant is empty and Q_max(b+1) there equals
    Q_max(b) here, so scale, zero-point and codes coincide."""
    rng = np.random.default_rng(b)
    for trial in range(10):
        m = np.abs(rng.standard_normal(257)).astype(np.float32)
        if trial % 2:
            m += np.float32(1.5)                                # non-zero minimum and zero-point
        m = raw_to_f32(f32_to_raw(m, R.BF16), R.BF16)
        s1, zp1, q1 = R.aiq_signed(m, b)
        s0, zp0, q0 = R.aiq(m, b + 1)
        assert (s1, zp1) == (s0, zp0) and np.array_equal(q1, q0)


def test_non_negative_blob_equals_the_magnitude_blob_without_its_sign_plane():
    rng = np.random.default_rng(11)
    T, H = 9, 100
    v = np.abs(rng.standard_normal((T, H)) * np.exp(rng.standard_normal((T, 1)))).astype(np.float32)
    v[2] = v[2] ** 4 * 0.01                                      # a row that descends
    v[rng.random((T, H)) < 0.02] *= 40
    raw = f32_to_raw(v, R.F16)
    a = R.encode(raw, R.F16, 6.0, [2, 3, 7], 0.2, signed_values=True)
    m = R.encode(raw, R.F16, 6.0, [3, 4, 8], 0.2)
    sa, sm = R.sections(a), R.sections(m)
    assert np.array_equal(sa["bits"] + 1, sm["bits"]) and len(set(sa["bits"].tolist())) > 1
    assert np.array_equal(sa["scale"], sm["scale"]) and np.array_equal(sa["zp"], sm["zp"])
    assert np.array_equal(sa["outl"], sm["outl"]) and np.array_equal(sa["out_ptr"], sm["out_ptr"])
    wpp = (H + 31) // 32
    for t in range(T):
        b = int(sa["bits"][t])
        wa = sa["words"][sa["word_off"][t]:sa["word_off"][t + 1]].reshape(wpp, b)
        wm = sm["words"][sm["word_off"][t]:sm["word_off"][t + 1]].reshape(wpp, b + 1)
        assert not wm[:, 0].any() and np.array_equal(wa, wm[:, 1:])
    assert np.array_equal(R.decode(a), R.decode(m))


# ---------------------------------------------------------------- closed form, bound, symmetry

@pytest.mark.parametrize("dtype", [R.F16, R.BF16])
@pytest.mark.parametrize("b", [2, 4, 8])
def test_affine_rounding_closed_form_and_error_bound(dtype, b):
    rng = np.random.default_rng(300 + b)
    qmax = 2 ** b - 1
    for trial in range(20):
        H = int(rng.integers(2, 300))
        v = (rng.standard_normal(H) * 10.0 ** rng.uniform(-3, 3)).astype(np.float32)
        if trial % 3 == 0:
            v += np.float32(rng.uniform(-50, 50))
        v = raw_to_f32(f32_to_raw(v, dtype), dtype)
        v = v[np.isfinite(v)]
        if v.size < 2 or v.max() == v.min():
            continue
        s, zp, q = R.aiq_signed(v, b)
        assert s == (np.float32(v.max()) - np.float32(v.min())) / np.float32(qmax)
        assert zp == int(torch.round(torch.tensor(np.float32(v.min()) / np.float32(s))).item())
        assert q.min() >= 0 and q.max() <= qmax
        # away from ties the code is round(v/s) - round(vmin/s) in exact arithmetic (a library rounding)
        t = v.astype(np.float64) / float(s)
        near_tie = np.abs(t - np.floor(t) - 0.5) < 1e-4 * (1 + np.abs(t))
        want = np.clip(torch.round(torch.from_numpy(t)).numpy().astype(np.int64) - zp, 0, qmax)
        assert np.array_equal(q[~near_tie], want[~near_tie])
        rec = (q.astype(np.float64) + zp) * float(s)
        slop = float(s) * (abs(zp) + qmax + 2) * 2.0 ** -22
        assert np.all(np.abs(rec - v.astype(np.float64)) <= float(s) / 2 + slop)
        assert q[np.argmin(v)] == 0 and q[np.argmax(v)] >= qmax - 1


def test_negated_row_mirrors_the_codes():
    """rint is odd, so negating the row maps code q to (rint(vmax/s) - rint(vmin/s)) - q before the clamp."""
    rng = np.random.default_rng(5)
    seen = 0
    for _ in range(50):
        v = raw_to_f32(f32_to_raw(rng.standard_normal(64).astype(np.float32), R.F16), R.F16)
        for b in (2, 3, 5, 8):
            s, zp, q = R.aiq_signed(v, b)
            s2, zp2, q2 = R.aiq_signed(-v, b)
            assert s2 == s
            span = int(np.rint(np.float32(v.max()) / np.float32(s))) - zp
            assert zp2 == -(zp + span)
            if span == 2 ** b - 1:                              # no clamp on either side
                assert np.array_equal(q2, span - q)
                seen += 1
    assert seen > 50


# ---------------------------------------------------------------- planes, restore, selection through the blob

def _indep_signed_codes(v32, b):
    qmax = np.float32(2 ** b - 1)
    lo, hi = np.float32(v32.min()), np.float32(v32.max())
    rng_ = np.float32(hi - lo)
    s = np.float32(rng_ / qmax) if rng_ > 0 else (np.float32(abs(hi)) if hi != 0 else np.float32(1))
    zp = int(np.rint(np.float32(lo / s)))
    q = np.rint((v32 / s).astype(np.float32)).astype(np.int64) - zp
    return np.clip(q, 0, int(qmax)), s, zp


@pytest.mark.parametrize("dtype", [R.F16, R.BF16])
@pytest.mark.parametrize("hidden", [1, 31, 33, 72, 200])
def test_blob_planes_restore_and_level_against_an_independent_reader(dtype, hidden):
    rng = np.random.default_rng(hidden + 7)
    T = 8
    v = (rng.standard_normal((T, hidden)) * np.exp(rng.standard_normal((T, 1)))).astype(np.float32)
    v[rng.random((T, hidden)) < 0.03] *= 30
    v[1] = np.sign(v[1]) * np.abs(v[1]) ** 4 * 0.01
    v[2] = -np.abs(v[2])                                         # an all-negative row
    raw = f32_to_raw(v, dtype)
    raw[3, 0] = 0x8000                                           # a -0 inlier decodes as what (code+zp)*s gives
    x = raw_to_f32(raw, dtype)
    bits, tau, delta = [2, 4, 8], 6.0, 0.2
    blob = R.encode(raw, dtype, tau, bits, delta, signed_values=True)
    hdr, sec = R.header(blob), R.sections(blob)
    assert hdr["variant"] == 1 and hdr["status"] == 0
    wpp = (hidden + 31) // 32
    assert sec["word_off"].tolist() == [0] + np.cumsum(sec["bits"].astype(np.int64) * wpp).tolist()
    out = ~(np.abs(x) < tau)
    y = R.decode(blob)
    for t in range(T):
        vt = np.where(out[t], np.float32(0), x[t]).astype(np.float32)
        # brute-force level: every candidate's distortion, stopping rule on exact rationals
        q0, _, _ = _indep_signed_codes(vt, 8)
        chosen = 8
        for b in (4, 2):
            q, _, _ = _indep_signed_codes(vt, b)
            if Fraction(int(np.abs((q0 >> (8 - b)) - q).sum()), hidden) > Fraction(float(np.float32(delta))):
                break
            chosen = b
        assert int(sec["bits"][t]) == chosen
        q, s, zp = _indep_signed_codes(vt, chosen)
        assert (np.float32(sec["scale"][t]), int(sec["zp"][t])) == (s, zp)
        words_row = sec["words"][sec["word_off"][t]:sec["word_off"][t + 1]]
        assert np.array_equal(codes_of_planes(words_row, chosen, hidden), q)
        if hidden % 32:
            mask = np.uint32((0xffffffff << (hidden % 32)) & 0xffffffff)
            assert np.all(words_row.reshape(wpp, chosen)[-1, :] & mask == 0)
        want = f32_to_raw(((q + zp).astype(np.float32) * s).astype(np.float32), dtype)
        want[out[t]] = raw[t][out[t]]
        assert np.array_equal(y[t], want)


def test_variant_flag_travels_and_bad_flag_is_rejected():
    raw = f16_raw([[1.0, -2.0, 3.0]])
    a = R.encode(raw, R.F16, INF, [8], signed_values=True)
    m = R.encode(raw, R.F16, INF, [8])
    assert R.header(a)["variant"] == 1 and R.header(m)["variant"] == 0
    bad = a.copy()
    bad[31] = 2
    with pytest.raises(R.OracleError) as e:
        R.decode(bad)
    assert e.value.status == 5
    # the same planes read under the other variant give another tensor: the flag is part of the format
    flipped = a.copy()
    flipped[31] = 0
    assert not np.array_equal(R.decode(flipped), R.decode(a))
