"""Exact-rational model of IEEE-754 binary64 arithmetic, for pinning the oracle's
double-precision gate.  Same conventions as ``tests/exact32.py`` (a ``Fraction`` for a
finite value, float ``inf``/``nan`` otherwise); every result is the exact real value
rounded to the nearest binary64 value (ties to even, gradual underflow, overflow to
infinity) by integer arithmetic written here, not by the machine's float unit.
"""
from __future__ import annotations

import struct
from fractions import Fraction

from tests.exact32 import INF, NAN, is_finite, is_inf, is_nan, fabs, le, lt, eq  # noqa: F401

_MAXFINITE = (Fraction(2) ** 53 - 1) * Fraction(2) ** 971          # DBL_MAX
_OVERFLOW = _MAXFINITE + Fraction(2) ** 970                        # halfway to 2^1024


def from_bits(u: int):
    sign = -1 if (u >> 63) & 1 else 1
    expo = (u >> 52) & 0x7FF
    frac = u & ((1 << 52) - 1)
    if expo == 0x7FF:
        return NAN if frac else sign * INF
    if expo == 0:
        return sign * Fraction(frac) * Fraction(2) ** -1074
    return sign * Fraction((1 << 52) + frac) * Fraction(2) ** (expo - 1075)


def from_float(f: float):
    return from_bits(struct.unpack("<Q", struct.pack("<d", f))[0])


def to_bits(x) -> int:
    """Model value (already a binary64 value) -> bit pattern; -0 is not represented."""
    if is_nan(x):
        return 0x7FF8000000000000
    if is_inf(x):
        return 0x7FF0000000000000 if x > 0 else 0xFFF0000000000000
    s = (1 << 63) if x < 0 else 0
    a = abs(x)
    if a == 0:
        return s
    e = a.numerator.bit_length() - a.denominator.bit_length()
    if Fraction(2) ** e > a:
        e -= 1
    if e < -1022:
        m = a / Fraction(2) ** -1074
        assert m.denominator == 1
        return s | int(m)
    m = a / Fraction(2) ** (e - 52)
    assert m.denominator == 1, "not a binary64 value"
    return s | ((e + 1023) << 52) | (int(m) - (1 << 52))


def rne(x):
    if not is_finite(x):
        return x
    if x == 0:
        return Fraction(0)
    sign = -1 if x < 0 else 1
    a = abs(x)
    if a >= _OVERFLOW:
        return sign * INF
    e = a.numerator.bit_length() - a.denominator.bit_length()
    if Fraction(2) ** e > a:
        e -= 1
    qe = max(e - 52, -1074)
    scaled = a / Fraction(2) ** qe
    m = scaled.numerator // scaled.denominator
    rem = scaled - m
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and (m & 1)):
        m += 1
    return sign * Fraction(m) * Fraction(2) ** qe


def sub(a, b):
    if is_nan(a) or is_nan(b):
        return NAN
    if is_inf(a) and is_inf(b):
        return NAN if a == b else a
    if is_inf(a):
        return a
    if is_inf(b):
        return -b
    return rne(a - b)


def add(a, b):
    if is_nan(a) or is_nan(b):
        return NAN
    if is_inf(a) and is_inf(b):
        return a if a == b else NAN
    if is_inf(a):
        return a
    if is_inf(b):
        return b
    return rne(a + b)


def mul(a, b):
    if is_nan(a) or is_nan(b):
        return NAN
    if is_inf(a) or is_inf(b):
        other = b if is_inf(a) else a
        if is_finite(other) and other == 0:
            return NAN
        sa = -1 if a < 0 else 1
        sb = -1 if b < 0 else 1
        return sa * sb * INF
    return rne(a * b)


def div(a, b):
    """a / b for b != 0."""
    if is_nan(a) or is_nan(b):
        return NAN
    if is_inf(a) and is_inf(b):
        return NAN
    if is_inf(a):
        return a if b > 0 else -a
    if is_inf(b):
        return Fraction(0)
    assert b != 0
    return rne(a / b)
