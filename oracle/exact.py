"""Exact rational arithmetic for pinning the oracle -- TEST INFRASTRUCTURE.

Nothing here uses floating-point arithmetic to decide a value: operands are converted to
``fractions.Fraction`` (every finite float is a rational), the operation is carried out exactly,
and the result is rounded once, to nearest with ties to even, into the target format by integer
arithmetic. Used on small inputs only (pure-Python loops).
"""
from __future__ import annotations

from fractions import Fraction

import numpy as np

# (significand bits incl. hidden bit, minimum normal exponent, maximum exponent)
_FORMATS = {"f64": (53, -1022, 1023), "f32": (24, -126, 127)}


def round_to_format(q: Fraction, fmt: str) -> float:
    """Round the rational ``q`` to the nearest ``fmt`` value, ties to even, with gradual
    underflow and overflow to infinity. Returns a Python float holding that value exactly."""
    p, emin, emax = _FORMATS[fmt]
    if q == 0:
        return 0.0
    sign = -1 if q < 0 else 1
    q = abs(q)
    # exponent e with 2**e <= q < 2**(e+1)
    e = q.numerator.bit_length() - q.denominator.bit_length()
    if Fraction(2) ** e > q:
        e -= 1
    elif Fraction(2) ** (e + 1) <= q:
        e += 1
    e = max(e, emin)                       # subnormals share the exponent of the smallest normal
    ulp = Fraction(2) ** (e - (p - 1))
    scaled = q / ulp                       # want the nearest integer, ties to even
    m = scaled.numerator // scaled.denominator
    rem = scaled - m
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and (m & 1)):
        m += 1
    val = Fraction(m) * ulp
    if val >= Fraction(2) ** (emax + 1):
        return sign * float("inf")
    return sign * float(val)               # exact: val is representable in fmt, hence in double


def fmt_of(arr: np.ndarray) -> str:
    return "f64" if arr.dtype == np.float64 else "f32"


def scalar_in_format(scalar: float, fmt: str) -> Fraction:
    """The scalar after its single rounding to the arrays' precision."""
    return Fraction(round_to_format(Fraction(float(scalar)), fmt))


def scale_exact(x: np.ndarray, scalar: float) -> np.ndarray:
    fmt = fmt_of(x)
    s = scalar_in_format(scalar, fmt)
    return np.array([round_to_format(s * Fraction(float(v)), fmt) for v in x], dtype=x.dtype)


def add_exact(x: np.ndarray, y: np.ndarray) -> np.ndarray:
    fmt = fmt_of(x)
    return np.array([round_to_format(Fraction(float(u)) + Fraction(float(v)), fmt)
                     for u, v in zip(x, y)], dtype=x.dtype)


def triad_exact(x: np.ndarray, y: np.ndarray, scalar: float) -> np.ndarray:
    """Two roundings: the product first, then the sum."""
    fmt = fmt_of(x)
    s = scalar_in_format(scalar, fmt)
    out = []
    for u, v in zip(x, y):
        prod = Fraction(round_to_format(s * Fraction(float(v)), fmt))
        out.append(round_to_format(Fraction(float(u)) + prod, fmt))
    return np.array(out, dtype=x.dtype)


def fma_exact(x: np.ndarray, y: np.ndarray, scalar: float) -> np.ndarray:
    """What a fused multiply-add would give (one rounding): the value Triad must NOT take."""
    fmt = fmt_of(x)
    s = scalar_in_format(scalar, fmt)
    return np.array([round_to_format(Fraction(float(u)) + s * Fraction(float(v)), fmt)
                     for u, v in zip(x, y)], dtype=x.dtype)


def dot_exact_fraction(x: np.ndarray, y: np.ndarray) -> Fraction:
    """The exact dot product as a rational (small n)."""
    acc = Fraction(0)
    for u, v in zip(x, y):
        acc += Fraction(float(u)) * Fraction(float(v))
    return acc


def dot_exact_bigint(x: np.ndarray, y: np.ndarray) -> Fraction:
    """The exact dot product through big-integer arithmetic: every finite float is m * 2**e with
    integer m, so the sum is an integer multiple of 2**(2*emin). Fast enough for n ~ 1e5."""
    total = 0
    shift = 2200                           # 2 * 1074 < 2200: makes every term an integer
    for u, v in zip(x.tolist(), y.tolist()):
        nu, du = float(u).as_integer_ratio()
        nv, dv = float(v).as_integer_ratio()
        # du, dv are powers of two
        total += (nu * nv) << (shift - (du.bit_length() - 1) - (dv.bit_length() - 1))
    return Fraction(total, 1 << shift)
