"""Exact-rational helpers for the oracle pins: one float32 rounding, and a fused
multiply-add chain evaluated with exactly one rounding per term. No numpy float
arithmetic is involved in the rounding, so the result cannot double-round."""
from fractions import Fraction

import numpy as np


def round_f32(q: Fraction) -> np.float32:
    """Round a rational to the nearest float32, ties to even (normal and subnormal range)."""
    if q == 0:
        return np.float32(0.0)
    sign = -1 if q < 0 else 1
    q = abs(q)
    e = q.numerator.bit_length() - q.denominator.bit_length()
    if Fraction(2) ** e > q:
        e -= 1
    e = max(e, -126)
    scaled = q / Fraction(2) ** (e - 23)  # significand as a rational in [2^23, 2^24)
    fl = scaled.numerator // scaled.denominator
    rem = scaled - fl
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2 == 1):
        fl += 1
    return np.float32(sign * float(Fraction(fl) * Fraction(2) ** (e - 23)))


def fma_chain_exact(ws, xs, b) -> np.float32:
    """acc = b; for each term: acc = float32(w * x + acc) with a single rounding."""
    acc = Fraction(float(b))
    for w, x in zip(ws, xs):
        acc = Fraction(float(round_f32(Fraction(float(w)) * Fraction(float(x)) + acc)))
    return np.float32(float(acc))


def chain_value(ws, xs, b) -> Fraction:
    """The same chain, returned as the exact rational value of its float32 result."""
    return Fraction(float(fma_chain_exact(ws, xs, b)))
