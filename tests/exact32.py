"""Exact-arithmetic model of IEEE binary32 operations, built on Python integers and
Fractions.  Used to pin the float32 steps of the oracle (division, multiplication,
subtraction, square root, round-to-integer) by a route that shares nothing with NumPy's
floating-point units: every result is the exact rational value rounded to the nearest
binary32 with ties to even."""
from decimal import Decimal, getcontext
from fractions import Fraction
import math
import struct


def f32_to_fraction(x):
    """Exact value of a binary32 given as a Python/NumPy float."""
    return Fraction(float(x))


def round_to_f32(q):
    """Nearest binary32 (ties to even) of the rational q, returned as a Fraction.
    Handles normals and subnormals; overflow is not expected in the tests."""
    q = Fraction(q)
    if q == 0:
        return Fraction(0)
    sign = -1 if q < 0 else 1
    a = abs(q)
    e = a.numerator.bit_length() - a.denominator.bit_length()
    if Fraction(2) ** e > a:
        e -= 1
    # now 2^e <= a < 2^(e+1)
    e = max(e, -126)
    ulp = Fraction(2) ** (e - 23)
    n = a / ulp
    lo = n.numerator // n.denominator
    rem = n - lo
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and lo % 2 == 1):
        lo += 1
    return sign * lo * ulp


def round_half_even_int(q):
    """Nearest integer, ties to even, of a rational."""
    q = Fraction(q)
    lo = q.numerator // q.denominator
    rem = q - lo
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and lo % 2 == 1):
        lo += 1
    return int(lo)


def sqrt_f32(q):
    """Correctly rounded binary32 square root of a positive rational (80-digit decimal
    square root, far beyond the 24-bit rounding boundary spacing)."""
    getcontext().prec = 80
    d = (Decimal(q.numerator) / Decimal(q.denominator)).sqrt()
    return round_to_f32(Fraction(d))


def fraction_bits(q):
    """Bit pattern (uint32) of a Fraction that is exactly a binary32."""
    return struct.unpack("<I", struct.pack("<f", float(q)))[0]


def quantize_row_exact(row, bits):
    """Codes and scale of one row under: s = fl(amax / qmax), code = clamp(rne(fl(w / s)))."""
    qmax = 2 ** (bits - 1) - 1
    vals = [f32_to_fraction(v) for v in row]
    amax = max(abs(v) for v in vals)
    s = round_to_f32(amax / qmax) if amax != 0 else Fraction(1)
    codes = []
    for v in vals:
        c = round_half_even_int(round_to_f32(v / s))
        codes.append(max(-(2 ** (bits - 1)), min(qmax, c)))
    return codes, s


def half_rne_exact(v):
    """Nearest IEEE half (ties to even) of a binary32 value, as a Fraction (normal and
    subnormal range; no overflow expected)."""
    q = f32_to_fraction(v)
    if q == 0:
        return Fraction(0)
    sign = -1 if q < 0 else 1
    a = abs(q)
    e = math.floor(math.log2(float(a)))
    while Fraction(2) ** e > a:
        e -= 1
    while Fraction(2) ** (e + 1) <= a:
        e += 1
    e = max(e, -14)
    ulp = Fraction(2) ** (e - 10)
    n = a / ulp
    lo = n.numerator // n.denominator
    rem = n - lo
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and lo % 2 == 1):
        lo += 1
    return sign * lo * ulp
