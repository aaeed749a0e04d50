"""Exact rational helpers for pinning the oracle: decode FP32 / BF16 bit patterns to Fractions and
round a Fraction to FP32 with round-to-nearest-even.  Written with integer arithmetic only, so it
is independent of the oracle's C++ and of the host's floating-point unit."""

from __future__ import annotations

import struct
from fractions import Fraction


def f32_bits(x: float) -> int:
    return struct.unpack("<I", struct.pack("<f", x))[0]


def bits_f32(b: int) -> float:
    return struct.unpack("<f", struct.pack("<I", b & 0xFFFFFFFF))[0]


def is_nan_bits(b: int) -> bool:
    return (b & 0x7FFFFFFF) > 0x7F800000


def is_inf_bits(b: int) -> bool:
    return (b & 0x7FFFFFFF) == 0x7F800000


def frac_of_f32_bits(b: int) -> Fraction:
    """Exact value of a finite FP32 pattern."""
    sign = -1 if b >> 31 else 1
    e = (b >> 23) & 0xFF
    man = b & 0x7FFFFF
    assert e != 0xFF, "not finite"
    if e == 0:
        return sign * Fraction(man, 1 << 149)
    return sign * Fraction((1 << 23) | man) * Fraction(2) ** (e - 150)


def frac_of_bf16_bits(h: int) -> Fraction:
    return frac_of_f32_bits((h & 0xFFFF) << 16)


def frac_of_float(x: float) -> Fraction:
    return frac_of_f32_bits(f32_bits(x))


_F32_MAX = frac_of_f32_bits(0x7F7FFFFF)
_F32_OVERFLOW = _F32_MAX + Fraction(2) ** 103  # half an ulp above FLT_MAX rounds to infinity


def round_to_f32_bits(q: Fraction, sign_of_zero: int = 0) -> int:
    """Correctly rounded (nearest, ties to even) FP32 pattern of an exact rational."""
    if q == 0:
        return 0x80000000 if sign_of_zero else 0
    sign = 0x80000000 if q < 0 else 0
    a = -q if q < 0 else q
    if a >= _F32_OVERFLOW:
        return sign | 0x7F800000
    # find e with 2^e <= a < 2^(e+1)
    e = a.numerator.bit_length() - a.denominator.bit_length()
    if Fraction(2) ** e > a:
        e -= 1
    elif Fraction(2) ** (e + 1) <= a:
        e += 1
    e = max(e, -126)                      # subnormals share the exponent of the smallest normal
    ulp = Fraction(2) ** (e - 23)
    scaled = a / ulp                      # in [2^23, 2^24) for normals, [0, 2^23) for subnormals
    n = scaled.numerator // scaled.denominator
    rem = scaled - n
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and (n & 1)):
        n += 1
    # n * ulp is the rounded magnitude; rebuild the pattern (carry into the exponent is automatic)
    if e == -126 and n < (1 << 23):
        return sign | n
    return sign | (((e + 127) << 23) + (n - (1 << 23)))


def round_to_f32(q: Fraction) -> float:
    return bits_f32(round_to_f32_bits(q))


def bf16_neighbours(fbits: int):
    """(lower, upper) BF16 patterns bracketing a finite non-NaN FP32 pattern in magnitude: lower is
    the truncation, upper is one BF16 step further from zero (equal to lower when exact)."""
    lo = fbits >> 16
    up = lo if (fbits & 0xFFFF) == 0 else lo + 1
    return lo, up
