"""Pins for the CPU oracle: everything here runs without a GPU and never touches the CUDA path.

Each test ties the oracle to something other than itself: hand-derived rows
(tests/golden/hand_rows.txt), identities the paper's equations fix, closed forms, library
conversions, error bounds, and brute-force enumeration written independently in numpy /
exact rationals.
"""
from fractions import Fraction
import math
import os

import numpy as np
import pytest
import torch

from oracle import tsq_ref as R

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
INF = float("inf")


def f16_raw(values):
    return torch.tensor(values, dtype=torch.float16).view(torch.int16).numpy().view(np.uint16)


def bf16_raw(values):
    return torch.tensor(values, dtype=torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def raw_to_f32(raw, dtype):
    t = torch.from_numpy(np.ascontiguousarray(raw).view(np.int16))
    t = t.view(torch.float16 if dtype == R.F16 else torch.bfloat16)
    return t.to(torch.float32).numpy()


def f32_to_raw(v, dtype):
    t = torch.from_numpy(np.ascontiguousarray(v, dtype=np.float32))
    t = t.to(torch.float16 if dtype == R.F16 else torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16)


def unpack_planes(words_row, b, hidden):
    """Independent scalar reader of one token's bit-planes: returns (sign[H], code[H]).
    Group g (elements 32g .. 32g+31) owns words g*b .. g*b+b-1: plane 0 = sign, plane 1+k = code bit k."""
    sign = np.zeros(hidden, np.int64)
    code = np.zeros(hidden, np.int64)
    for j in range(hidden):
        g, i = divmod(j, 32)
        sign[j] = (int(words_row[g * b]) >> i) & 1
        c = 0
        for k in range(b - 1):
            c |= ((int(words_row[g * b + 1 + k]) >> i) & 1) << k
        code[j] = c
    return sign, code


# ---------------------------------------------------------------- 16-bit conversions vs a library

@pytest.mark.parametrize("dtype", [R.F16, R.BF16])
def test_raw16_to_float_all_patterns(dtype):
    raw = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    want = raw_to_f32(raw, dtype)
    got = np.array([R.raw16_to_float(dtype, int(r)) for r in raw], dtype=np.float32)
    assert np.array_equal(got.view(np.uint32)[~np.isnan(want)], want.view(np.uint32)[~np.isnan(want)])
    assert np.all(np.isnan(got[np.isnan(want)]))


@pytest.mark.parametrize("dtype", [R.F16, R.BF16])
def test_float_to_raw16_rne(dtype):
    rng = np.random.default_rng(7)
    # every 16-bit value, the midpoints between neighbours (ties) and points just off them
    raw = np.arange(0, 0x7c00 if dtype == R.F16 else 0x7f80, dtype=np.uint32).astype(np.uint16)
    v = raw_to_f32(raw, dtype).astype(np.float64)
    mids = (v[:-1] + v[1:]) / 2
    cand = np.concatenate([v, mids, np.nextafter(mids.astype(np.float32), np.float32(0)).astype(np.float64),
                           np.nextafter(mids.astype(np.float32), np.float32(np.inf)).astype(np.float64),
                           rng.standard_normal(20000) * 10.0 ** rng.uniform(-9, 5, 20000),
                           [65519.99, 65520.0, 65536.0, 1e30, 3.4e38, 1e-40, 1e-45, 0.0]])
    cand = np.abs(cand).astype(np.float32)
    cand = np.concatenate([cand, -cand])
    want = f32_to_raw(cand, dtype)
    got = np.array([R.float_to_raw16(dtype, float(c)) for c in cand], dtype=np.uint16)
    assert np.array_equal(got, want)


# ---------------------------------------------------------------- hand-derived rows

def _hand_rows():
    rows = []
    with open(os.path.join(GOLDEN, "hand_rows.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            p = [s.strip() for s in line.split("|")]
            rows.append(dict(m=[float(v) for v in p[0].split()], bits=[int(v) for v in p[1].split()],
                             delta=float(p[2]), b=int(p[3]), s=float(p[4]), zp=int(p[5]),
                             codes=[int(v) for v in p[6].split()], recon=[float(v) for v in p[7].split()]))
    return rows


@pytest.mark.parametrize("row", _hand_rows(), ids=lambda r: "%s-%s-%g" % (r["m"], r["bits"], r["delta"]))
@pytest.mark.parametrize("negate", [False, True])
def test_hand_rows(row, negate):
    vals = [-v for v in row["m"]] if negate else row["m"]
    x = f16_raw([vals])
    blob = R.encode(x, R.F16, INF, row["bits"], row["delta"])
    sec = R.sections(blob)
    H = len(vals)
    assert sec["bits"].tolist() == [row["b"]]
    assert sec["scale"][0] == np.float32(row["s"])
    assert sec["zp"].tolist() == [row["zp"]]
    sign, code = unpack_planes(sec["words"], row["b"], H)
    assert code.tolist() == row["codes"]
    # the sign plane is the raw sign bit (a negated zero keeps it)
    assert sign.tolist() == [1 if negate else 0] * H
    y = raw_to_f32(R.decode(blob), R.F16)[0]
    want = np.array(row["recon"], dtype=np.float32) * (-1 if negate else 1)
    assert np.array_equal(y, want)
    assert np.array_equal(np.signbit(y), np.signbit(np.array(vals, dtype=np.float32)))


# ---------------------------------------------------------------- TS: Eq. "ts"

@pytest.mark.parametrize("dtype", [R.F16, R.BF16])
def test_ts_is_exact_partition(dtype):
    rng = np.random.default_rng(11)
    v = (rng.standard_normal(4096) * 3).astype(np.float32)
    v[:6] = [6.0, -6.0, 5.996, np.inf, -np.inf, np.nan]
    raw = f32_to_raw(v, dtype)
    x = raw_to_f32(raw, dtype)
    tau = 6.0
    m, sg, is_out, n_out = R.ts_row(raw, dtype, tau)
    want_out = ~(np.abs(x) < tau)                       # |T| >= tau, and NaN
    assert np.array_equal(is_out.astype(bool), want_out)
    assert is_out[0] == 1 and is_out[1] == 1            # |x| == tau is an outlier (>=)
    assert n_out == int(want_out.sum())
    # T_below = T * (1 - M): magnitude and sign of the inliers, +0 in outlier slots
    assert np.array_equal(m[~want_out], np.abs(x[~want_out]))
    assert np.all(m[want_out] == 0) and not np.any(np.signbit(m[want_out]))
    assert np.array_equal(sg[~want_out].astype(bool), np.signbit(x[~want_out]))
    assert np.all(sg[want_out] == 0)
    # T_above + T_below = T on the finite entries
    below = np.where(sg.astype(bool), -m, m)
    above = np.where(want_out, x, 0.0)
    fin = np.isfinite(x)
    assert np.array_equal((above + below)[fin], x[fin])


def test_ts_outlier_fraction_matches_gaussian_tail():
    rng = np.random.default_rng(5)
    v = rng.standard_normal(1 << 20).astype(np.float32)
    raw = f32_to_raw(v, R.BF16)
    tau = 2.0
    _, _, _, n_out = R.ts_row(raw, R.BF16, tau)
    p = math.erfc(tau / math.sqrt(2))                   # 2 * (1 - Phi(tau))
    n = v.size
    assert abs(n_out - n * p) < 6 * math.sqrt(n * p) + n * 2 ** -8 * 0.12  # + bf16 rounding at the edge


@pytest.mark.parametrize("dtype", [R.F16, R.BF16])
def test_outliers_survive_bit_exactly_and_csr_is_sorted(dtype):
    rng = np.random.default_rng(3)
    T, H = 5, 200
    v = rng.standard_normal((T, H)).astype(np.float32)
    v[rng.random((T, H)) < 0.05] *= 40
    v[0, 7] = np.nan
    v[1, 0] = np.inf
    v[2, H - 1] = -np.inf
    raw = f32_to_raw(v, dtype)
    x = raw_to_f32(raw, dtype)
    tau = 5.0
    blob = R.encode(raw, dtype, tau, [2, 4, 8], 0.2)
    sec, hdr = R.sections(blob), R.header(blob)
    y = R.decode(blob)
    out = ~(np.abs(x) < tau)
    assert np.array_equal(y[out], raw[out])             # transmitted without distortion
    # CSR: row pointers are the prefix sums of the per-row counts, columns ascend within a row
    counts = out.sum(axis=1)
    assert sec["out_ptr"].tolist() == [0] + np.cumsum(counts).tolist()
    assert hdr["total_outliers"] == int(out.sum())
    for t in range(T):
        e = sec["outl"][sec["out_ptr"][t]:sec["out_ptr"][t + 1]]
        cols = (e >> 16).astype(np.int64)
        assert np.array_equal(cols, np.nonzero(out[t])[0])
        assert np.array_equal((e & 0xffff).astype(np.uint16), raw[t][out[t]])


# ---------------------------------------------------------------- AIQ: Eq. "Proposed"

@pytest.mark.parametrize("b", [2, 3, 4, 5, 8])
def test_aiq_reduces_to_absmax_rounding_when_min_is_zero(b):
    """With m_min = 0 the scheme is textbook abs-max quantisation q = round(m * Qmax / max m)."""
    rng = np.random.default_rng(b)
    m = np.abs(rng.standard_normal(2000)).astype(np.float32)
    m[0] = 0.0
    m = raw_to_f32(f32_to_raw(m, R.F16), R.F16)
    qmax = 2 ** (b - 1) - 1
    s, zp, q = R.aiq(m, b)
    assert zp == 0
    assert s == np.float32(m.max()) / np.float32(qmax)
    exact = m.astype(np.float64) * qmax / float(m.max())
    want = torch.round(torch.from_numpy(exact)).numpy().astype(np.int64)     # ties-to-even, a library routine
    near_tie = np.abs(exact - np.floor(exact) - 0.5) < 1e-5
    assert np.array_equal(q[~near_tie], want[~near_tie])
    assert np.all(np.abs(q[near_tie] - exact[near_tie]) <= 0.5 + 1e-5)
    assert q.min() == 0 and q.max() == qmax


@pytest.mark.parametrize("dtype", [R.F16, R.BF16])
@pytest.mark.parametrize("b", [2, 4, 8])
def test_aiq_error_bound_and_code_range(dtype, b):
    rng = np.random.default_rng(100 + b)
    for trial in range(20):
        H = int(rng.integers(1, 300))
        m = np.abs(rng.standard_normal(H) * 10.0 ** rng.uniform(-3, 3)).astype(np.float32)
        if trial % 3 == 0:
            m += np.float32(rng.uniform(0, 50))          # non-zero minimum -> non-zero zero-point
        m = raw_to_f32(f32_to_raw(m, dtype), dtype)
        m = m[np.isfinite(m)]
        if m.size == 0:
            continue
        qmax = 2 ** (b - 1) - 1
        s, zp, q = R.aiq(m, b)
        assert q.min() >= 0 and q.max() <= qmax
        rec = (q.astype(np.float64) + zp) * float(s)
        slop = float(s) * (abs(zp) + qmax + 2) * 2.0 ** -22
        assert np.all(np.abs(rec - m.astype(np.float64)) <= float(s) / 2 + slop)
        if m.max() > m.min():
            assert s == (np.float32(m.max()) - np.float32(m.min())) / np.float32(qmax)
            assert zp == int(torch.round(torch.tensor(np.float32(m.min()) / np.float32(s))).item())


def test_aiq_degenerate_ranges():
    s, zp, q = R.aiq(np.zeros(17, np.float32), 4)
    assert (s, zp, q.tolist()) == (1.0, 0, [0] * 17)
    s, zp, q = R.aiq(np.full(9, 2.5, np.float32), 8)
    assert (s, zp, q.tolist()) == (2.5, 1, [0] * 9)     # restore (0 + 1) * 2.5 = 2.5 exactly
    s, zp, q = R.aiq(np.array([3.0], np.float32), 2)
    assert (s, zp, q.tolist()) == (3.0, 1, [0])


# ---------------------------------------------------------------- Algorithm 1: level selection

def _indep_codes(m32, b):
    """AIQ restated with numpy binary32 scalars (a different code path from the oracle's C++)."""
    qmax = np.float32(2 ** (b - 1) - 1)
    lo, hi = np.float32(m32.min()), np.float32(m32.max())
    rng_ = np.float32(hi - lo)
    s = np.float32(rng_ / qmax) if rng_ > 0 else (hi if hi > 0 else np.float32(1))
    zp = int(np.rint(np.float32(lo / s)))
    q = np.rint((m32 / s).astype(np.float32)).astype(np.int64) - zp
    return np.clip(q, 0, int(qmax)), s, zp


def _brute_force_level(m32, bits, delta32):
    """Enumerate every candidate's distortion, then apply the stopping rule on exact rationals."""
    bmax = bits[-1]
    q0, _, _ = _indep_codes(m32, bmax)
    n = m32.size
    S = {}
    for b in bits[:-1]:
        q, _, _ = _indep_codes(m32, b)
        S[b] = int(np.abs((q0 >> (bmax - b)) - q).sum())
    chosen = bmax
    for b in reversed(bits[:-1]):
        if Fraction(S[b], n) > Fraction(float(np.float32(delta32))):   # delta > Delta, exactly
            break
        chosen = b
    return chosen, S


@pytest.mark.parametrize("bits", [[2, 4, 8], [2, 3, 4, 8], [2, 3, 4, 5, 6, 7, 8], [3, 4], [5]])
def test_selection_matches_brute_force_on_tiny_rows(bits):
    rng = np.random.default_rng(sum(bits))
    deltas = [-1.0, 0.0, 0.05, 0.2, 0.25, 0.5, 1.0, 3.0, 1e9]
    for trial in range(150):
        H = int(rng.integers(1, 24))
        kind = trial % 4
        if kind == 0:
            m = np.abs(rng.standard_normal(H))
        elif kind == 1:
            m = rng.integers(0, 9, H) / 2.0             # many exact ties
        elif kind == 2:
            m = np.abs(rng.standard_normal(H)) ** 4      # bulk small against the range
        else:
            m = np.abs(rng.standard_normal(H)) + 3.0
        m32 = raw_to_f32(f32_to_raw(m.astype(np.float32), R.F16), R.F16)
        for d in deltas:
            S, b_star = R.select(m32, bits, d)
            want_b, want_S = _brute_force_level(m32, bits, d)
            assert S[:-1] == [want_S[b] for b in bits[:-1]]
            assert b_star == want_b, (m32, bits, d, S)


def test_selection_limits_and_monotonicity():
    rng = np.random.default_rng(2)
    bits = [2, 3, 4, 6, 8]
    for _ in range(40):
        m = raw_to_f32(f32_to_raw(np.abs(rng.standard_normal(64)).astype(np.float32), R.BF16), R.BF16)
        assert R.select(m, bits, 1e9)[1] == bits[0]      # nothing ever fails -> lowest candidate
        assert R.select(m, bits, -1.0)[1] == bits[-1]    # everything fails -> top level
        assert R.select(m, [4], 0.2)[1] == 4             # single candidate
        prev = bits[-1]
        for d in [0.0, 0.1, 0.2, 0.5, 1.0, 2.0, 5.0, 50.0]:
            b = R.select(m, bits, d)[1]
            assert b <= prev                             # b*(Delta) never increases with Delta
            prev = b
    assert R.select(np.zeros(32, np.float32), bits, 0.0)[1] == bits[0]   # all-zero row: S = 0 everywhere


# ---------------------------------------------------------------- layout, offsets, restore

@pytest.mark.parametrize("dtype", [R.F16, R.BF16])
@pytest.mark.parametrize("hidden", [1, 31, 32, 33, 72, 200])
def test_blob_layout_offsets_and_restore(dtype, hidden):
    rng = np.random.default_rng(hidden)
    T = 6
    scale_t = np.exp(rng.standard_normal((T, 1)))
    v = (rng.standard_normal((T, hidden)) * scale_t).astype(np.float32)
    v[rng.random((T, hidden)) < 0.02] *= 30
    v[1] = np.abs(v[1]) ** 4 * 0.01                      # a row that drops to a low level
    raw = f32_to_raw(v, dtype)
    x = raw_to_f32(raw, dtype)
    bits = [2, 4, 8]
    tau = 6.0
    blob = R.encode(raw, dtype, tau, bits, 0.2)
    hdr, sec = R.header(blob), R.sections(blob)
    wpp = (hidden + 31) // 32
    assert (hdr["magic"], hdr["version"], hdr["dtype"], hdr["hidden"], hdr["tokens"]) == \
        (int.from_bytes(b"TSQ1", "little"), 1, dtype, hidden, T)
    assert hdr["bits"][:3] == bits and hdr["n_bits"] == 3 and hdr["status"] == 0
    # placement is a plain exclusive prefix sum of bits * WPP
    assert sec["word_off"].tolist() == [0] + np.cumsum(sec["bits"].astype(np.int64) * wpp).tolist()
    assert hdr["total_words"] == int(sec["word_off"][-1])
    lay = R.layout(hidden, T, 8, 0)
    for name in ("bits", "scale", "zp", "word_off", "out_ptr", "words", "outl", "total"):
        assert lay[name] % 16 == 0
    assert lay["total"] == blob.size
    # restore each row with an independent reader: (code + zp) * s, one rounding to 16 bits, sign, outliers
    y = R.decode(blob)
    out = ~(np.abs(x) < tau)
    for t in range(T):
        b = int(sec["bits"][t])
        assert b in bits
        words_row = sec["words"][sec["word_off"][t]:sec["word_off"][t + 1]]
        sign, code = unpack_planes(words_row, b, hidden)
        assert code.max() <= 2 ** (b - 1) - 1
        assert np.all(code[out[t]] == 0) and np.all(sign[out[t]] == 0)
        mag = ((code + int(sec["zp"][t])).astype(np.float32) * np.float32(sec["scale"][t])).astype(np.float32)
        want = f32_to_raw(mag, dtype) | (sign.astype(np.uint16) << 15)
        want[out[t]] = raw[t][out[t]]
        assert np.array_equal(y[t], want)
        # pad bits of the last word are zero in every plane
        if hidden % 32:
            mask = np.uint32((0xffffffff << (hidden % 32)) & 0xffffffff)
            assert np.all(words_row.reshape(wpp, b)[-1, :] & mask == 0)
        # inlier error bound after the cast: s/2 + half a 16-bit ulp of the restored value
        inl = ~out[t]
        s = float(sec["scale"][t])
        yv = raw_to_f32(y[t], dtype).astype(np.float64)
        ulp = np.abs(yv) * 2.0 ** (-10 if dtype == R.F16 else -7) + 2.0 ** -24
        with np.errstate(invalid="ignore"):
            err = np.abs(yv - x[t].astype(np.float64))
        assert np.all(err[inl] <= s / 2 + ulp[inl] / 2 + s * 2.0 ** -12)


def test_empty_and_all_outlier_and_signed_zero():
    blob = R.encode(np.zeros((0, 64), np.uint16), R.F16, 6.0, [2, 4, 8])
    hdr = R.header(blob)
    assert hdr["tokens"] == 0 and hdr["total_words"] == 0 and hdr["total_outliers"] == 0
    assert R.decode(blob).shape == (0, 64)
    # tau <= 0: every element is an outlier, so the round trip is the identity and codes are all zero
    rng = np.random.default_rng(0)
    raw = f32_to_raw(rng.standard_normal((3, 50)).astype(np.float32), R.BF16)
    blob = R.encode(raw, R.BF16, 0.0, [2, 4, 8])
    sec = R.sections(blob)
    assert R.header(blob)["total_outliers"] == 150
    assert sec["bits"].tolist() == [2, 2, 2] and not sec["words"].any()
    assert np.array_equal(R.decode(blob), raw)
    # -0.0 keeps its sign; subnormal rows survive without flush-to-zero
    raw = f16_raw([[-0.0, 0.0, 1.0, -1.0], [6e-8, -1.2e-7, 0.0, 1.8e-7]])
    y = R.decode(R.encode(raw, R.F16, INF, [8]))
    assert y[0].tolist() == raw[0].tolist()
    assert y[1].tolist() == raw[1].tolist()             # 3 subnormal steps fit 127 levels exactly


def test_outlier_capacity_overflow_is_reported_not_written():
    raw = f16_raw([[10.0, 1.0, 20.0, 30.0], [40.0, 0.5, 0.25, 50.0]])
    blob = R.encode(raw, R.F16, 6.0, [4], 0.2, max_outliers=3)
    hdr = R.header(blob)
    assert hdr["status"] == 6 and hdr["total_outliers"] == 5 and hdr["outlier_capacity"] == 3
    sec = R.sections(blob)
    assert sec["out_ptr"].tolist() == [0, 3, 5] and sec["outl"].size == 3
    with pytest.raises(R.OracleError) as e:
        R.decode(blob)
    assert e.value.status == 6


def test_argument_errors():
    raw = np.zeros((2, 8), np.uint16)
    for bad_bits in ([], [1, 4], [4, 4], [4, 2], [2, 9], list(range(2, 9)) + [8]):
        with pytest.raises(R.OracleError):
            R.encode(raw, R.F16, 6.0, bad_bits)
    with pytest.raises(R.OracleError):
        R.encode(raw, R.F16, float("nan"), [2, 4])
    with pytest.raises(R.OracleError):
        R.encode(raw, 2, 6.0, [2, 4])
    blob = R.encode(raw, R.F16, 6.0, [2, 4])
    bad = blob.copy()
    bad[0] ^= 0xff
    with pytest.raises(R.OracleError) as e:
        R.decode(bad)
    assert e.value.status == 5
