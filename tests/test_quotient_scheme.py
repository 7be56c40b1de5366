"""The division-free quotient of the CUDA encoder, checked on the host in exact arithmetic.

The kernels form rint(m / s) for "plain" rows as  q0 = fl(m r), e = fl(m - q0 s) (one FMA), q = fl(q0 + e r)
(one FMA), rint(q)  with r = fl(1 / s), instead of the IEEE quotient the method is defined with.  This test
restates that three-operation sequence with exactly rounded binary32 steps (fractions, then one rounding per
step) and compares rint against rint of the correctly rounded quotient, for every non-negative 16-bit magnitude
below the row's maximum, over many (maximum, level) pairs of both 16-bit types, adversarial ones included."""
from fractions import Fraction

import numpy as np
import pytest


def f32(fr: Fraction) -> Fraction:
    """Round a non-negative rational to the nearest binary32 (ties to even); normal range only."""
    if fr == 0:
        return Fraction(0)
    e = fr.numerator.bit_length() - fr.denominator.bit_length()
    if Fraction(2) ** e > fr:
        e -= 1
    if Fraction(2) ** (e + 1) <= fr:
        e += 1
    q = Fraction(2) ** (e - 23)                      # unit in the last place
    n = fr / q
    k = n.numerator // n.denominator
    rem = n - k
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and (k & 1)):
        k += 1
    return k * q


def f32_signed(fr: Fraction) -> Fraction:
    return f32(fr) if fr >= 0 else -f32(-fr)


def rint(fr: Fraction) -> int:
    k = fr.numerator // fr.denominator
    rem = fr - k
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and (k & 1)):
        k += 1
    return k


def pattern_value(p: int, bf16: bool) -> Fraction:
    if bf16:
        e, f = (p >> 7) & 0xff, p & 0x7f
        return Fraction(f, 128) * Fraction(2) ** (-126) if e == 0 else (1 + Fraction(f, 128)) * Fraction(2) ** (e - 127)
    e, f = (p >> 10) & 0x1f, p & 0x3ff
    return Fraction(f, 1024) * Fraction(2) ** (-14) if e == 0 else (1 + Fraction(f, 1024)) * Fraction(2) ** (e - 15)


def check_row(pmax: int, bf16: bool, b: int, patterns) -> None:
    qmax = (1 << (b - 1)) - 1
    mmax = pattern_value(pmax, bf16)
    s = f32(mmax / qmax)                               # minimum 0: range = max
    r = f32(1 / s)
    for p in patterns:
        m = pattern_value(p, bf16)
        want = rint(f32(m / s))
        q0 = f32(m * r)
        e = f32_signed(m - q0 * s)
        q = f32_signed(q0 + e * r)
        assert rint(q) == want, (pmax, bf16, b, p, float(m), float(s))
        assert 0 <= want <= qmax


@pytest.mark.parametrize("bf16", [False, True])
def test_fma_quotient_equals_the_ieee_quotient_after_rint(bf16):
    rng = np.random.default_rng(7 if bf16 else 11)
    lo, hi = (0x3800, 0x4900) if bf16 else (0x2400, 0x5400)     # maxima between about 2^-15 / 2^-6 and 2^19 / 64
    maxima = sorted(set(rng.integers(lo, hi, 24).tolist() + [lo, hi - 1, 0x3f80 if bf16 else 0x3c00,
                                                             0x40e0 if bf16 else 0x4700, 0x4100 if bf16 else 0x4800]))
    for pmax in maxima:
        for b in (2, 3, 4, 8):
            # every pattern of the top three binades (where codes change most often), a sample of the rest
            step = 0x80 if bf16 else 0x400
            dense = range(max(1, pmax - 3 * step), pmax + 1)
            sparse = rng.integers(1, max(2, pmax - 3 * step), 200).tolist() if pmax > 3 * step + 2 else []
            check_row(pmax, bf16, b, list(dense) + sparse)


def check_signed_row(pmin: int, pmax: int, bf16: bool, b: int, patterns) -> int:
    """The signed-values variant's fast steps on a row that spans [-value(pmin), +value(pmax)]: the same three
    operations on the signed value, rounding by adding 2^23 + 2^22, the code as the low byte of the sum's integer
    minus the zero-point, modulo 256.  Returns how many patterns were checked (rows that are not plain: 0)."""
    qmax = (1 << b) - 1
    vmin, vmax = -pattern_value(pmin, bf16), pattern_value(pmax, bf16)
    s = f32(f32(vmax - vmin) / qmax)
    r = f32(1 / s)
    zp = rint(f32_signed(vmin / s))
    if rint(f32_signed(vmax / s)) - zp > qmax:
        return 0                                        # a code would need the clamp: such a level takes the division instruction
    magic = Fraction(12582912)
    n = 0
    for sign, bound in ((1, pmax), (-1, pmin)):
        for p in patterns:
            if p > bound:
                continue
            v = sign * pattern_value(p, bf16)
            want = rint(f32_signed(v / s)) - zp
            assert 0 <= want <= qmax
            q0 = f32_signed(v * r)
            e = f32_signed(v - q0 * s)
            q = f32_signed(q0 + e * r)
            t = f32_signed(q + magic)
            assert t.denominator == 1 and Fraction(2) ** 23 <= t < Fraction(2) ** 24
            low22 = (int(t) - (1 << 23)) & 0x3fffff        # the pattern's low mantissa bits: 2^22 + k
            assert ((low22 & 0xff) - (zp & 0xff)) & 0xff == want, (pmin, pmax, bf16, b, sign, p)
            n += 1
    return n


@pytest.mark.parametrize("bf16", [False, True])
def test_signed_values_fast_steps(bf16):
    rng = np.random.default_rng(17 if bf16 else 19)
    lo, hi = (0x3c00, 0x4600) if bf16 else (0x3000, 0x5000)
    checked = 0
    for _ in range(10):
        pmin, pmax = int(rng.integers(lo, hi)), int(rng.integers(lo, hi))
        for b in (2, 4, 8):
            top = max(pmin, pmax)
            step = 0x80 if bf16 else 0x400
            dense = list(range(max(1, top - 2 * step), top + 1))
            sparse = rng.integers(0, max(2, top - 2 * step), 150).tolist()
            checked += check_signed_row(pmin, pmax, bf16, b, dense + sparse)
    assert checked > 5000
