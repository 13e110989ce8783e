"""Shared test utilities: exact rational rounding, ulp distance, bit views.

None of these call the oracle or the CUDA library; they are the independent
yardsticks both are measured with.
"""
from __future__ import annotations

from fractions import Fraction

import numpy as np


def f32_from_fraction(x: Fraction) -> np.float32:
    """Correctly rounded (nearest, ties-to-even) fp32 value of a rational."""
    if x == 0:
        return np.float32(0.0)
    sign = -1 if x < 0 else 1
    a = -x if x < 0 else x
    # exponent e with 2^e <= a < 2^(e+1)
    e = a.numerator.bit_length() - a.denominator.bit_length()
    if Fraction(2) ** e > a:
        e -= 1
    elif Fraction(2) ** (e + 1) <= a:
        e += 1
    e = max(e, -126)                      # denormals share the 2^-149 quantum
    quantum = Fraction(2) ** (e - 23)
    q = a / quantum
    n = q.numerator // q.denominator
    rem = q - n
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and (n & 1)):
        n += 1
    val = n * quantum
    if val >= Fraction(2) ** 128:
        return np.float32(sign * np.inf)
    return np.float32(sign * float(val))  # exact: val is an fp32 number


def ordered_int(a: np.ndarray) -> np.ndarray:
    """Monotone integer image of fp32 values (+0 and -0 both map to 0)."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.int32).astype(np.int64)
    return np.where(u < 0, -(u & 0x7FFFFFFF), u)


def ulp_distance(a: np.ndarray, b: np.ndarray) -> np.ndarray:
    """Units in the last place between two fp32 arrays (NaN/Inf must agree)."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    b = np.ascontiguousarray(b, dtype=np.float32)
    fin_a, fin_b = np.isfinite(a), np.isfinite(b)
    d = np.abs(ordered_int(a) - ordered_int(b))
    bad = fin_a != fin_b
    both_nonfinite = ~fin_a & ~fin_b
    same_special = both_nonfinite & ((np.isnan(a) & np.isnan(b)) | (a == b))
    d = np.where(both_nonfinite, np.where(same_special, 0, 1 << 40), d)
    return np.where(bad, 1 << 40, d)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns (uint16) to fp32 by the defining shift."""
    return (bits.astype(np.uint32) << 16).view(np.float32)


def is_bf16_nan(bits: np.ndarray) -> np.ndarray:
    b = bits.astype(np.uint32)
    return ((b & 0x7F80) == 0x7F80) & ((b & 0x007F) != 0)
