"""Exact-arithmetic helpers for pinning fp32 results (no numpy float ops).

``round_f32`` rounds a rational number to the nearest IEEE-754 binary32 value,
ties to even, with gradual underflow, using integer arithmetic only.  It lets a
test state what "one correctly rounded operation" must give without trusting
any floating-point unit.
"""
from __future__ import annotations

import struct
from fractions import Fraction


def f32_to_fraction(x) -> Fraction:
    """Exact value of a (finite) binary32 number given as Python/numpy float."""
    return Fraction(float(x))


def round_f32(q: Fraction) -> float:
    """Nearest binary32 to the rational q (ties to even); returns a Python float."""
    if q == 0:
        return 0.0
    sign = -1 if q < 0 else 1
    a = abs(q)
    # exponent e with 2^e <= a < 2^(e+1)
    e = a.numerator.bit_length() - a.denominator.bit_length()
    if Fraction(2) ** e > a:
        e -= 1
    elif Fraction(2) ** (e + 1) <= a:
        e += 1
    e = max(e, -126)                  # subnormal range shares the exponent -126
    ulp = Fraction(2) ** (e - 23)
    n = a / ulp                       # significand in units of one ulp
    lo = n.numerator // n.denominator
    rem = n - lo
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and lo % 2 == 1):
        lo += 1
    val = lo * ulp
    if val >= Fraction(2) ** 128:
        return sign * float("inf")
    return sign * float(val)


def f32_bits(x: float) -> int:
    return struct.unpack("<I", struct.pack("<f", x))[0]


def ulp_distance(a: float, b: float) -> int:
    """Distance in units in the last place between two finite binary32 values."""
    def key(v):
        u = f32_bits(v)
        return -(u & 0x7FFFFFFF) if u >> 31 else u
    return abs(key(a) - key(b))
