"""An integer model of IEEE-754 binary32 arithmetic for the oracle's pins.

Every fp32 operation is "the exact result, rounded to the nearest fp32, ties to
even".  Here the exact result is a Python Fraction and the rounding is done with
integer arithmetic only, so a chain of such operations can be modelled without
touching the machine's float unit.  Used to pin the operation sequence of the
oracle's bin index (the shared bins of Sec. 3.3) at and next to the bin edges,
and to show which other plausible sequences give a different bin there.
Holds none of the oracle's or the library's code.
"""
import math
import struct
from fractions import Fraction

F32_MAX = Fraction((1 << 24) - 1) * Fraction(2) ** 104


def frac_of_f32(x) -> Fraction:
    """Exact rational value of a finite fp32 number, from its bit pattern."""
    bits = struct.unpack("<I", struct.pack("<f", float(x)))[0]
    sign = -1 if bits >> 31 else 1
    e = (bits >> 23) & 0xFF
    m = bits & 0x7FFFFF
    assert e != 0xFF, "not finite"
    if e == 0:
        return sign * Fraction(m, 1 << 149)
    return sign * Fraction((1 << 23) | m, 1) * Fraction(2) ** (e - 150)


def round_to_precision(q: Fraction, bits: int, e_min: int) -> Fraction:
    """q rounded to the nearest number with a `bits`-bit significand (ties to even) and
    exponent >= e_min (gradual underflow); no overflow handling."""
    if q == 0:
        return Fraction(0)
    s = -1 if q < 0 else 1
    a = abs(q)
    e = a.numerator.bit_length() - a.denominator.bit_length()
    if Fraction(2) ** e > a:
        e -= 1
    if Fraction(2) ** (e + 1) <= a:
        e += 1
    assert Fraction(2) ** e <= a < Fraction(2) ** (e + 1)
    e = max(e, e_min)
    ulp = Fraction(2) ** (e - (bits - 1))
    k = a / ulp
    lo = k.numerator // k.denominator
    rem = k - lo
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and (lo & 1)):
        lo += 1
    return s * lo * ulp


def rn32(q: Fraction) -> Fraction:
    """One fp32 rounding (finite results only)."""
    r = round_to_precision(q, 24, -126)
    assert abs(r) <= F32_MAX, "overflow is outside this model"
    return r


def rn64(q: Fraction) -> Fraction:
    """One fp64 rounding."""
    return round_to_precision(q, 53, -1022)


def bin_separate_fp32_ops(v: Fraction, lo: Fraction, hi: Fraction, n_bins: int) -> int:
    """The reading taken for the shared bins: w = hi - lo; scale = n_bins / w; t = v - lo;
    u = t * scale; floor; clamp - each a separate fp32 operation."""
    w = rn32(hi - lo)
    if w == 0:
        return 0
    scale = rn32(Fraction(n_bins) / w)
    t = rn32(v - lo)
    u = rn32(t * scale)
    return min(max(math.floor(u), 0), n_bins - 1)


# Other sequences a reader could plausibly have written; each differs from the reading above only
# for values within a rounding error of a bin edge.

def bin_product_unrounded(v, lo, hi, n_bins):
    """t * scale kept exact (an evaluation in double, or a product fused into what follows)."""
    w = rn32(hi - lo)
    if w == 0:
        return 0
    scale = rn32(Fraction(n_bins) / w)
    t = rn32(v - lo)
    return min(max(math.floor(t * scale), 0), n_bins - 1)


def bin_divide_then_multiply(v, lo, hi, n_bins):
    """(v - lo) / w * n_bins instead of (v - lo) * (n_bins / w)."""
    w = rn32(hi - lo)
    if w == 0:
        return 0
    t = rn32(v - lo)
    u = rn32(rn32(t / w) * n_bins)
    return min(max(math.floor(u), 0), n_bins - 1)


def bin_all_double(v, lo, hi, n_bins):
    """Every step in fp64."""
    w = rn64(hi - lo)
    if w == 0:
        return 0
    scale = rn64(Fraction(n_bins) / w)
    t = rn64(v - lo)
    u = rn64(t * scale)
    return min(max(math.floor(u), 0), n_bins - 1)


def bin_exact(v, lo, hi, n_bins):
    """The real-number definition floor((v - lo) n_bins / (hi - lo))."""
    if hi == lo:
        return 0
    return min(max(math.floor((v - lo) * n_bins / (hi - lo)), 0), n_bins - 1)


VARIANTS = {"product_unrounded": bin_product_unrounded,
            "divide_then_multiply": bin_divide_then_multiply,
            "all_double": bin_all_double,
            "exact": bin_exact}
