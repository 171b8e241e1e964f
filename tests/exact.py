"""Exact-rational helpers for the checker's pins: correct rounding of a Fraction to
IEEE binary32 (round-to-nearest-even), independent of any hardware float unit."""
from fractions import Fraction
import struct


def f32_to_fraction(x) -> Fraction:
    return Fraction(float(x))  # a float32 value is exactly representable as a double


def round_to_f32(v: Fraction) -> float:
    """Nearest binary32 (ties to even) of an exact rational; returns a Python float."""
    if v == 0:
        return 0.0
    sign = -1 if v < 0 else 1
    a = abs(v)
    # find e with 2^e <= a < 2^(e+1)
    e = a.numerator.bit_length() - a.denominator.bit_length()
    if Fraction(2) ** e > a:
        e -= 1
    elif Fraction(2) ** (e + 1) <= a:
        e += 1
    e_min = -126
    q_exp = max(e, e_min) - 23           # exponent of one unit in the last place
    scaled = a / (Fraction(2) ** q_exp)
    m = scaled.numerator // scaled.denominator
    rem = scaled - m
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and (m & 1)):
        m += 1
    val = Fraction(m) * (Fraction(2) ** q_exp)
    if val >= Fraction(2) ** 128:
        return sign * float("inf")
    return sign * float(val)


def f32_bits(x: float) -> int:
    return struct.unpack("<I", struct.pack("<f", x))[0]
