"""Software FP8 (OCP E4M3 / E5M2) for the oracle.  Test infrastructure only.

The paper casts activations and weights to E4M3 and gradients to E5M2 (Sec. 2.1,
"Temporal Latency and Hidden State in Delayed Scaling", citing the OCP FP8
formats) and leaves the conversion to its backend.  The reading used here:
round to nearest, ties to even, saturate to the largest finite value; NaN maps
to the format's canonical NaN; the sign of zero is kept.

Everything is written from the definition of the formats:
  value(code) = (-1)^s * 2^(max(E,1) - bias) * (M / 2^m + [E > 0])
with E4M3: 4 exponent bits, 3 mantissa bits, bias 7, no infinities, only
S.1111.111 is NaN (largest finite 448 = 0x7E); E5M2: 5 exponent bits, 2 mantissa
bits, bias 15, IEEE-style Inf/NaN in the top exponent (largest finite 57344 =
0x7B).  Encoding is "nearest representable value, ties to the even code",
decided by comparing with the exact midpoint of the two neighbouring codes.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


@dataclass(frozen=True)
class FP8Format:
    name: str
    exp_bits: int
    man_bits: int
    bias: int
    max_code: int  # code of the largest finite positive value
    nan_code: int  # canonical positive NaN

    @property
    def max_finite(self) -> float:
        return float(decode_code(self.max_code, self))


def decode_code(code: int, fmt: FP8Format) -> float:
    """Value of one 8-bit code by the format definition (NaN/Inf included)."""
    s = (code >> 7) & 1
    e = (code >> fmt.man_bits) & ((1 << fmt.exp_bits) - 1)
    m = code & ((1 << fmt.man_bits) - 1)
    sign = -1.0 if s else 1.0
    top = (1 << fmt.exp_bits) - 1
    if fmt.name == "e4m3":
        if e == top and m == (1 << fmt.man_bits) - 1:
            return float("nan")
    else:
        if e == top:
            return sign * float("inf") if m == 0 else float("nan")
    if e == 0:
        return sign * (m / (1 << fmt.man_bits)) * 2.0 ** (1 - fmt.bias)
    return sign * (1.0 + m / (1 << fmt.man_bits)) * 2.0 ** (e - fmt.bias)


E4M3 = FP8Format("e4m3", 4, 3, 7, 0x7E, 0x7F)
E5M2 = FP8Format("e5m2", 5, 2, 15, 0x7B, 0x7F)


def _tables(fmt: FP8Format):
    """Positive finite values in code order (code k holds values[k]) and all-256 decode table."""
    pos = np.array([decode_code(c, fmt) for c in range(fmt.max_code + 1)], dtype=np.float64)
    full = np.array([decode_code(c, fmt) for c in range(256)], dtype=np.float64)
    return pos, full


_POS = {f.name: _tables(f)[0] for f in (E4M3, E5M2)}
_FULL = {f.name: _tables(f)[1] for f in (E4M3, E5M2)}


def decode(codes: np.ndarray, fmt: FP8Format) -> np.ndarray:
    """uint8 codes -> float64 values (exact)."""
    codes = np.asarray(codes, dtype=np.uint8)
    return _FULL[fmt.name][codes]


_BLOCK = 1 << 18  # elements handled at a time by encode()


def encode(values: np.ndarray, fmt: FP8Format) -> np.ndarray:
    """float32 values -> uint8 codes, element by element (see _encode_block).

    The map is elementwise, so the tensor is walked in blocks of 2^18 elements
    only to keep the float64 / int64 temporaries of a block small; the result
    does not depend on the block size (full-size test tensors have 10^8
    elements, and whole-tensor temporaries of a gigabyte each made the cast
    six times slower without changing a bit of it).
    """
    v = np.ascontiguousarray(values, dtype=np.float32)
    if v.size <= _BLOCK:
        return _encode_block(v, fmt)
    flat = v.reshape(-1)
    out = np.empty(flat.size, dtype=np.uint8)
    for lo in range(0, flat.size, _BLOCK):
        out[lo : lo + _BLOCK] = _encode_block(flat[lo : lo + _BLOCK], fmt)
    return out.reshape(v.shape)


def _encode_block(values: np.ndarray, fmt: FP8Format) -> np.ndarray:
    """Round to nearest even, saturate to finite.

    For a magnitude a: find neighbouring codes lo <= a <= hi among the positive
    finite values; pick lo if a is below their midpoint, hi if above, and the
    even code on an exact tie.  Magnitudes at or above the largest finite value
    (Inf included) give that value.  The sign bit is the input's sign bit.
    """
    v = np.asarray(values, dtype=np.float32)
    pos = _POS[fmt.name]
    a = np.abs(v).astype(np.float64)
    nan = np.isnan(a)
    a_safe = np.where(nan, 0.0, a)
    # index of the first table entry strictly greater than a; lo is the one before it
    hi_idx = np.searchsorted(pos, a_safe, side="right")
    lo_idx = hi_idx - 1  # pos[0] = 0 <= a always, so lo_idx >= 0
    sat = hi_idx > fmt.max_code  # a >= largest finite
    hi_idx_c = np.minimum(hi_idx, fmt.max_code)
    lo = pos[lo_idx]
    hi = pos[hi_idx_c]
    mid = (lo + hi) * 0.5  # exact: both have at most 4 significant bits
    choose_hi = (a_safe > mid) | ((a_safe == mid) & ((lo_idx & 1) == 1))
    code = np.where(choose_hi, hi_idx_c, lo_idx)
    code = np.where(sat, fmt.max_code, code)
    code = np.where(nan, fmt.nan_code, code)
    sign = np.signbit(v).astype(np.int64) << 7
    return (code.astype(np.int64) | sign).astype(np.uint8)


def quantize(x_f32: np.ndarray, scale: np.float32, fmt: FP8Format) -> np.ndarray:
    """Cast step of delayed scaling: one IEEE fp32 multiply by the scale, then encode().

    The product is rounded to fp32 before the FP8 rounding (two roundings); that
    double rounding is part of the definition, so it is reproduced rather than
    rounding once from a wider type.
    """
    x = np.asarray(x_f32, dtype=np.float32)
    if x.size > _BLOCK:  # elementwise, so block by block (see encode); same bits as the whole tensor at once
        flat = np.ascontiguousarray(x).reshape(-1)
        out = np.empty(flat.size, dtype=np.uint8)
        for lo in range(0, flat.size, _BLOCK):
            out[lo : lo + _BLOCK] = quantize(flat[lo : lo + _BLOCK], scale, fmt)
        return out.reshape(x.shape)
    with np.errstate(over="ignore", invalid="ignore"):
        prod = x * np.float32(scale)  # numpy keeps float32 * float32 in float32 (IEEE RN)
    assert prod.dtype == np.float32
    return encode(prod, fmt)
