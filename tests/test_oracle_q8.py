"""Pins for the oracle's 8-bit code of retained values: exact rational arithmetic, an independent numpy statement of
the rounding, closed-form properties (round trip of codes, error bound, monotonicity, saturation)."""
from fractions import Fraction

import numpy as np
import pytest

import oracle


def _value(bits: int) -> Fraction:
    sign = -1 if bits & 0x8000 else 1
    e, m = (bits >> 7) & 0xFF, bits & 0x7F
    if e == 0:
        return sign * Fraction(m) * Fraction(1, 2 ** 133)
    return sign * Fraction(128 + m) * Fraction(2) ** (e - 134)


def _code_value(c: int, e_top: int) -> Fraction:
    u = Fraction(2) ** (e_top - 137)
    c &= 0x7F
    e, m = c >> 4, c & 15
    return m * u if e == 0 else (16 + m) * Fraction(2) ** (e - 1) * u


@pytest.mark.parametrize("e_top", [11, 100, 127, 129, 254])
def test_codes_round_trip_and_decode_is_the_stated_value(e_top):
    codes = np.arange(256, dtype=np.uint8)
    vals = oracle.q8_decode(codes, e_top)
    for c in range(256):
        exp = _code_value(c, e_top) * (-1 if c & 0x80 else 1)
        assert _value(int(vals[c])) == exp
        assert (int(vals[c]) >> 15) == (c >> 7)                      # the sign survives on zero too
    back = oracle.q8_encode(vals, e_top)
    assert (back == codes).all()


@pytest.mark.parametrize("e_top", [127, 130])
def test_encode_is_nearest_code_ties_to_even_against_exact_arithmetic(e_top):
    grid = [_code_value(c, e_top) for c in range(128)]
    bits = np.arange(0x7F80, dtype=np.uint16)                          # every finite non-negative bf16 pattern
    got = oracle.q8_encode(bits, e_top)
    for b in range(0, 0x7F80, 5):
        v = _value(b)
        if v >= grid[127]:
            exp = 127
        else:
            lo = max(c for c in range(128) if grid[c] <= v)
            hi = lo + 1
            dl, dh = v - grid[lo], grid[hi] - v
            exp = lo if dl < dh else hi if dh < dl else (lo if lo % 2 == 0 else hi)
        assert int(got[b]) == exp, (hex(b), int(got[b]), exp)
    # monotone in the magnitude, sign carried over
    assert (np.diff(got.astype(np.int32)) >= 0).all()
    neg = oracle.q8_encode(bits | np.uint16(0x8000), e_top)
    assert (neg == (got | 0x80)).all()


def test_error_bound_saturation_and_special_patterns():
    rng = np.random.default_rng(0)
    # retained values of N(0,1) at gamma = 0.9: |x| >= 1.64
    x = rng.standard_normal(200_000).astype(np.float32)
    x = x[np.abs(x) > 1.6449]
    bits = (x.view(np.uint32) >> 16).astype(np.uint16)
    e_top = oracle.q8_top_exponent(bits)
    assert e_top == int(((bits >> 7) & 0xFF).max())
    dec = oracle.q8_decode(oracle.q8_encode(bits, e_top), e_top)
    v = (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    d = (dec.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    assert (np.abs(d - v) <= np.abs(v) / 32 + 1e-300).all()
    assert np.abs(d - v).max() > 0                                         # it does round
    # Inf, NaN and values above the scale saturate to the largest code; zero and tiny values become signed zero
    assert list(oracle.q8_encode(np.array([0x7F80, 0xFF80, 0x7FC1, 0x4400], np.uint16), 127)) == [0x7F, 0xFF, 0x7F, 0x7F]
    assert list(oracle.q8_encode(np.array([0x0000, 0x8000, 0x0001, 0x3000], np.uint16), 127)) == [0x00, 0x80, 0x00, 0x00]
    assert oracle.q8_top_exponent(np.array([0x7F80, 0x7FC0, 0x3F80], np.uint16)) == 127      # non-finite values do not set the scale
    assert (oracle.q8_encode(np.array([0x3F80], np.uint16), 5) == 0).all()                     # no usable scale


def test_encode_against_numpy_rint():
    """The same rounding written with numpy: |v| / u rounded by np.rint in the binade's step."""
    e_top = 128
    bits = np.arange(0x7F80, dtype=np.uint16)
    v = (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    a = np.ldexp(v, 137 - e_top)
    e = np.where(a < 16, 0, np.floor(np.log2(np.maximum(a, 1))).astype(np.int64) - 3)
    step = np.where(e == 0, 1.0, np.ldexp(1.0, np.maximum(e - 1, 0)))
    code = np.where(e == 0, np.rint(a), (np.maximum(e, 1) - 1) * 16 + np.rint(a / step))
    code = np.minimum(code, 127).astype(np.uint8)
    assert (oracle.q8_encode(bits, e_top) == code).all()
