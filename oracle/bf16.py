"""bfloat16 bit helpers for the oracle.  Test infrastructure only.

bfloat16 is the top 16 bits of an IEEE binary32: 1 sign, 8 exponent, 7 mantissa
bits.  Tensors cross the oracle's boundary as uint16 bit patterns so that no
library's bfloat16 type (and its rounding) is involved.
"""
from __future__ import annotations

import numpy as np


def decode(bits: np.ndarray) -> np.ndarray:
    """uint16 bfloat16 bit patterns -> float32 values (exact)."""
    b = np.asarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << 16).view(np.float32)


def round_from_f64(v: np.ndarray) -> np.ndarray:
    """float64 -> nearest bfloat16 (ties to even), returned as uint16 bits.  One rounding.

    A bfloat16 has 8 significant bits.  For v = m * 2^e with 0.5 <= |m| < 1 the
    spacing of bfloat16 values around v is 2^(e-8), but never finer than the
    subnormal spacing 2^-133.  v is scaled by that spacing (exact: a power of
    two), rounded half-to-even to an integer, and scaled back.
    """
    v = np.asarray(v, dtype=np.float64)
    _, e = np.frexp(v)
    ulp_exp = np.maximum(e.astype(np.int64) - 8, -133)
    with np.errstate(over="ignore", invalid="ignore"):
        q = np.ldexp(np.rint(np.ldexp(v, -ulp_exp)), ulp_exp)
        # q has at most 8 significant bits, so float32 holds it exactly; values past the
        # largest bfloat16 (2^128 after rounding) become Inf in float32, as they should.
        f = q.astype(np.float32)
    f = np.where(np.isfinite(v), f, v.astype(np.float32))
    return (f.view(np.uint32) >> 16).astype(np.uint16)


def ulp(v: np.ndarray) -> np.ndarray:
    """Spacing of bfloat16 values at magnitude |v| (float64)."""
    v = np.abs(np.asarray(v, dtype=np.float64))
    _, e = np.frexp(v)
    e = np.where(v == 0, -(1 << 20), e.astype(np.int64))  # frexp(0) reports exponent 0; zero sits among the subnormals
    return np.ldexp(1.0, np.maximum(e - 8, -133))
