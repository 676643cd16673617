"""Shared test utilities: exact-rational helpers and bf16 distance. No method arithmetic of the
CUDA path or of the oracle lives here."""
from fractions import Fraction

import numpy as np


def f32_frac(v) -> Fraction:
    return Fraction(float(np.float32(v)))


def round_frac_to_f32(fr: Fraction) -> np.float32:
    """Correctly rounded (nearest, ties to even) float32 of an exact rational."""
    c = np.float32(float(fr))  # within a couple of ulps; refine exactly
    cands = {c, np.nextafter(c, np.float32(np.inf)), np.nextafter(c, np.float32(-np.inf))}
    best = None
    for v in cands:
        d = abs(Fraction(float(v)) - fr)
        even = (np.float32(v).view(np.uint32) & 1) == 0
        key = (d, 0 if even else 1)
        if best is None or key < best[0]:
            best = (key, v)
    return np.float32(best[1])


def bf16_bits(vals) -> np.ndarray:
    """bf16 bit patterns of values that are exactly representable in bf16."""
    f = np.asarray(vals, np.float32)
    u = f.view(np.uint32)
    assert np.all((u & 0xFFFF) == 0), "value not representable in bf16"
    return (u >> 16).astype(np.uint16)


def bf16_ordinal(bits: np.ndarray) -> np.ndarray:
    """Monotone integer mapping of bf16 bit patterns (distance 1 = adjacent values)."""
    b = bits.astype(np.int32)
    return np.where(b & 0x8000, -(b & 0x7FFF), b & 0x7FFF)


def bf16_ulp_dist(a: np.ndarray, b: np.ndarray) -> np.ndarray:
    return np.abs(bf16_ordinal(a) - bf16_ordinal(b))
