"""Pins for the oracle's statement of the producer in front of the path (Sec. 3.5: the activation whose output is
the conv / fc input): the bf16 rounding, the activation tables and the key histogram are checked against things
that are not the oracle itself (exact rational arithmetic, scipy's erf, closed forms, numpy's bincount)."""
import math
from fractions import Fraction

import numpy as np
import pytest
import scipy.special

import oracle


def _bf16_value(bits: int) -> Fraction:
    """Exact value of a finite bf16 bit pattern."""
    sign = -1 if bits & 0x8000 else 1
    e, m = (bits >> 7) & 0xFF, bits & 0x7F
    if e == 0:
        return sign * Fraction(m, 1) * Fraction(1, 2 ** 133)
    return sign * Fraction(128 + m, 1) * (Fraction(2) ** (e - 127 - 7))


def _round_exact(v: Fraction, negative_zero: bool = False) -> int:
    """Round an exact rational to bf16 bits, ties to even, by searching the finite positive patterns."""
    sign = 0x8000 if (v < 0 or (v == 0 and negative_zero)) else 0
    a = abs(v)
    lo, hi = 0, 0x7F80          # patterns are monotone in value; 0x7F80 stands for 2^128
    top = Fraction(2) ** 128
    val = lambda b: top if b == 0x7F80 else _bf16_value(b)
    while hi - lo > 1:
        mid = (lo + hi) // 2
        if val(mid) <= a:
            lo = mid
        else:
            hi = mid
    if a >= top:
        return sign | 0x7F80
    dl, dh = a - val(lo), val(hi) - a
    if dl < dh:
        r = lo
    elif dh < dl:
        r = hi
    else:
        r = lo if lo % 2 == 0 else hi
    return sign | r


def test_round_to_bf16_matches_exact_rational_rounding():
    rng = np.random.default_rng(0)
    vals = list(rng.standard_normal(300) * 10.0 ** rng.integers(-42, 39, 300))
    # ties and near-ties that a rounding through fp32 would get wrong, the subnormal range, the overflow boundary
    vals += [1.0 + 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -40, 1.0 + 3 * 2.0 ** -8, 1.0 + 3 * 2.0 ** -8 - 2.0 ** -45,
             2.0 ** -133, 2.0 ** -134, 3 * 2.0 ** -134, 2.0 ** -126, 2.0 ** -126 - 2.0 ** -134, 127.5 * 2.0 ** -133,
             float(np.finfo(np.float32).max), 3.3961775292304304e38, 3.39e38, 3.4e38, 1e-45, 0.0, -0.0, -1.5]
    for v in vals:
        for s in (1.0, -1.0):
            x = s * float(v)
            got = oracle.round_to_bf16(x)
            exp = _round_exact(Fraction(x), negative_zero=math.copysign(1.0, x) < 0)
            assert got == exp, (x, hex(got), hex(exp))
    assert oracle.round_to_bf16(float("inf")) == 0x7F80 and oracle.round_to_bf16(float("-inf")) == 0xFF80
    assert oracle.round_to_bf16(float("nan")) == 0x7FC0


def test_relu_and_identity_tables_in_closed_form():
    b = np.arange(65536, dtype=np.uint32)
    ident = oracle.activation_table(oracle.ACT_IDENTITY)
    assert (ident == b).all()
    relu = oracle.activation_table(oracle.ACT_RELU)
    key = b & 0x7FFF
    nan = key > 0x7F80
    neg = (b & 0x8000) != 0
    exp = np.where(nan, b, np.where(neg, 0, b)).astype(np.uint16)       # -x and -0 -> +0, NaN passes, +x stays
    assert (relu == exp).all()
    assert relu[0x8000] == 0 and relu[0xFF80] == 0 and relu[0x7F80] == 0x7F80


def test_gelu_table_against_an_independent_erf_and_exact_rounding():
    table = oracle.activation_table(oracle.ACT_GELU)
    b = np.arange(65536, dtype=np.uint32)
    key = b & 0x7FFF
    # NaN in, the same NaN out; -Inf -> the one NaN pattern; +Inf stays
    assert (table[key > 0x7F80] == b[key > 0x7F80]).all()
    assert table[0x7F80] == 0x7F80 and table[0xFF80] == 0x7FC0
    assert table[0] == 0 and table[0x8000] == 0x8000                    # 0.5 * (+-0) * 1
    finite = np.flatnonzero(key < 0x7F80)
    x = (finite.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    phi = 0.5 * (1.0 + scipy.special.erf(x / math.sqrt(2.0)))            # scipy's erf, not libm's
    # where 1 + erf cancels badly (x << 0) use erfc: Phi(x) = erfc(-x / sqrt 2) / 2, accurate in the tail
    phi = np.where(x < -1.0, 0.5 * scipy.special.erfc(-x / math.sqrt(2.0)), phi)
    y = x * phi
    mismatches = 0
    for i in range(0, finite.size, 7):                                   # every 7th pattern: ~9300 exact roundings
        exp = _round_exact(Fraction(float(y[i])), negative_zero=math.copysign(1.0, float(y[i])) < 0)
        got = int(table[finite[i]])
        if got != exp:
            # the two erf implementations may differ in the last bits of a double; that can only matter within
            # a hair of a rounding boundary, and then the two candidates are neighbours
            assert abs((got & 0x7FFF) - (exp & 0x7FFF)) <= 1, (hex(int(finite[i])), hex(got), hex(exp))
            mismatches += 1
    assert mismatches <= 3
    # shape of the function: x for large x, -0 or a vanishing negative number for very negative x, x / 2 near 0
    assert table[0x4200] == 0x4200                                       # gelu(32) = 32
    assert table[0xC2C8] == 0x8000                                       # gelu(-100) underflows to -0
    assert table[0xC100] == _round_exact(Fraction(-8.0) * Fraction(float(0.5 * scipy.special.erfc(8.0 / math.sqrt(2.0)))))
    assert table[0x3800] == 0x3780                                       # gelu(2^-15) = 2^-16
    pos = table[0x3F80:0x4180].astype(np.int64)                          # monotone for x >= 1
    assert (np.diff(pos) >= 0).all()


def test_apply_table_and_key_histogram():
    rng = np.random.default_rng(3)
    x = rng.integers(0, 65536, 100_000).astype(np.uint16)
    table = oracle.activation_table(oracle.ACT_GELU)
    y = oracle.apply_table(table, x)
    assert (y == table[x]).all()
    h = oracle.key_histogram_bf16(y)
    assert (h == np.bincount(y & 0x7FFF, minlength=32768)).all()
    assert int(h.sum()) == x.size
