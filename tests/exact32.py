"""Exact-rational model of IEEE-754 binary32 arithmetic, for pinning the oracle.

Values are Python objects: a ``Fraction`` for finite numbers, ``INF``/``-INF``
(floats) for infinities and ``NAN`` for NaN.  Every operation computes the
exact real result with ``fractions.Fraction`` and then rounds to the nearest
binary32 value (ties to even, gradual underflow, overflow to infinity) with
integer arithmetic written here -- it does not use the machine's float unit, so
it cannot share a mistake with compiled C code.  Only for tiny inputs.
"""
from __future__ import annotations

import math
import struct
from fractions import Fraction

INF = float("inf")
NAN = float("nan")

_TWO = Fraction(2)
_MAXFINITE = (Fraction(2) ** 24 - 1) * Fraction(2) ** 104          # FLT_MAX
_OVERFLOW = _MAXFINITE + Fraction(2) ** 103                        # halfway to 2^128


def is_nan(x) -> bool:
    return isinstance(x, float) and math.isnan(x)


def is_inf(x) -> bool:
    return isinstance(x, float) and math.isinf(x)


def is_finite(x) -> bool:
    return isinstance(x, Fraction)


def from_bits(u: int):
    """binary32 bit pattern -> model value."""
    sign = -1 if (u >> 31) & 1 else 1
    expo = (u >> 23) & 0xFF
    frac = u & 0x7FFFFF
    if expo == 0xFF:
        return NAN if frac else sign * INF
    if expo == 0:
        return sign * Fraction(frac) * Fraction(2) ** -149
    return sign * Fraction((1 << 23) + frac) * Fraction(2) ** (expo - 150)


def from_float(f: float):
    return from_bits(struct.unpack("<I", struct.pack("<f", f))[0])


def to_bits(x) -> int:
    """Model value (already a binary32 value) -> bit pattern; -0 is not represented."""
    if is_nan(x):
        return 0x7FC00000
    if is_inf(x):
        return 0x7F800000 if x > 0 else 0xFF800000
    s = 0x80000000 if x < 0 else 0
    a = abs(x)
    if a == 0:
        return s
    e = a.numerator.bit_length() - a.denominator.bit_length()
    if Fraction(2) ** e > a:
        e -= 1
    if e < -126:
        m = a / Fraction(2) ** -149
        assert m.denominator == 1
        return s | int(m)
    m = a / Fraction(2) ** (e - 23)
    assert m.denominator == 1, "not a binary32 value"
    return s | ((e + 127) << 23) | (int(m) - (1 << 23))


def rne(x):
    """Round an exact value to binary32 (nearest, ties to even)."""
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
    assert Fraction(2) ** e <= a < Fraction(2) ** (e + 1)
    qe = max(e - 23, -149)
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
    """a / b for b != 0 (the screen never divides by zero)."""
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


def fabs(a):
    if is_nan(a):
        return NAN
    return abs(a)


def le(a, b) -> bool:
    if is_nan(a) or is_nan(b):
        return False
    return a <= b


def lt(a, b) -> bool:
    if is_nan(a) or is_nan(b):
        return False
    return a < b


def eq(a, b) -> bool:
    if is_nan(a) or is_nan(b):
        return False
    return a == b
