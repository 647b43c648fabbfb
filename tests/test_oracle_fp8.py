"""Pins for the oracle's FP8 and bf16 encoders (CPU only)."""
import os
from fractions import Fraction

import ml_dtypes
import numpy as np
import pytest
import torch

from oracle import bf16, fp8

GOLD = os.path.join(os.path.dirname(__file__), "golden")
FMT = {"e4m3": fp8.E4M3, "e5m2": fp8.E5M2}


def _boundary_rows():
    rows = []
    for line in open(os.path.join(GOLD, "fp8_boundary_codes.txt")):
        line = line.split("#")[0].strip()
        if not line:
            continue
        parts = line.split()
        # the value expression may contain no spaces except inside float('inf'); re-join until hex
        fmt, expr, code = parts[0], parts[1], parts[2]
        rows.append((fmt, expr, int(code, 16)))
    return rows


@pytest.mark.parametrize("fmt,expr,code", _boundary_rows())
def test_hand_computed_codes(fmt, expr, code):
    v = np.float32(eval(expr))
    assert int(fp8.encode(np.array([v]), FMT[fmt])[0]) == code


@pytest.mark.parametrize("fmt", ["e4m3", "e5m2"])
def test_decode_encode_round_trip_all_codes(fmt):
    f = FMT[fmt]
    codes = np.arange(256, dtype=np.uint8)
    vals = fp8.decode(codes, f)
    finite = np.isfinite(vals)
    back = fp8.encode(vals[finite].astype(np.float32), f)
    assert np.array_equal(back, codes[finite])
    # format facts
    assert f.max_finite == (448.0 if fmt == "e4m3" else 57344.0)
    n_nan = int(np.isnan(vals).sum())
    n_inf = int(np.isinf(vals).sum())
    assert (n_nan, n_inf) == ((2, 0) if fmt == "e4m3" else (6, 2))


@pytest.mark.parametrize("fmt", ["e4m3", "e5m2"])
def test_decode_matches_exact_rational_definition(fmt):
    f = FMT[fmt]
    for c in range(f.max_code + 1):
        e = (c >> f.man_bits) & ((1 << f.exp_bits) - 1)
        m = c & ((1 << f.man_bits) - 1)
        if e == 0:
            exact = Fraction(m, 1 << f.man_bits) * Fraction(2) ** (1 - f.bias)
        else:
            exact = (1 + Fraction(m, 1 << f.man_bits)) * Fraction(2) ** (e - f.bias)
        assert Fraction(float(fp8.decode(np.uint8(c), f))) == exact
        assert Fraction(float(fp8.decode(np.uint8(c | 0x80), f))) == -exact


@pytest.mark.parametrize("fmt", ["e4m3", "e5m2"])
def test_every_midpoint_rounds_to_even_and_neighbours_round_nearest(fmt):
    f = FMT[fmt]
    for c in range(f.max_code):
        lo, hi = float(fp8.decode(np.uint8(c), f)), float(fp8.decode(np.uint8(c + 1), f))
        mid = np.float32((lo + hi) / 2)
        assert float(mid) == (lo + hi) / 2  # representable
        even = c if c % 2 == 0 else c + 1
        assert int(fp8.encode(np.array([mid]), f)[0]) == even
        assert int(fp8.encode(np.array([-mid]), f)[0]) == even | 0x80
        below = np.nextafter(mid, np.float32(0))
        above = np.nextafter(mid, np.float32(np.inf))
        assert int(fp8.encode(np.array([below]), f)[0]) == c
        assert int(fp8.encode(np.array([above]), f)[0]) == c + 1


@pytest.mark.parametrize("fmt,ml", [("e4m3", ml_dtypes.float8_e4m3fn), ("e5m2", ml_dtypes.float8_e5m2)])
def test_agrees_with_library_cast_inside_finite_range(fmt, ml):
    f = FMT[fmt]
    rng = np.random.default_rng(7)
    # log-uniform magnitudes across the whole range incl. subnormals, random signs, plus exact grid points
    mag = np.exp2(rng.uniform(-20, np.log2(f.max_finite), size=200_000)).astype(np.float32)
    v = mag * rng.choice([-1.0, 1.0], size=mag.size).astype(np.float32)
    v = v[np.abs(v) <= f.max_finite]
    ours = fp8.encode(v, f)
    lib = v.astype(ml).view(np.uint8)
    assert np.array_equal(ours, lib)


def test_nan_maps_to_canonical_nan():
    assert int(fp8.encode(np.array([np.nan], np.float32), fp8.E4M3)[0]) & 0x7F == 0x7F
    assert int(fp8.encode(np.array([np.nan], np.float32), fp8.E5M2)[0]) & 0x7F == 0x7F


def test_quantize_exact_products_match_hand_codes():
    # scale a power of two -> product exact -> bytes follow from the boundary table
    x = np.array([0.25, 0.015625, 108.0, 200.0, -112.0], np.float32)  # *4 -> 1, 0.0625, 432, 800, -448
    q = fp8.quantize(x, np.float32(4.0), fp8.E4M3)
    assert [int(b) for b in q] == [0x38, 0x18, 0x7E, 0x7E, 0xFE]


def test_quantize_double_rounding_is_reproduced():
    # x*scale lands, after fp32 rounding, exactly on an FP8 tie although the real product is above it
    scale = np.float32(1.0 + 2.0**-23)
    x = np.float32(1.0625)  # exact product 1.0625*(1+2^-23) > tie 1.0625; fp32 product rounds...
    prod32 = np.float32(x * scale)
    exact = Fraction(float(x)) * Fraction(float(scale))
    code = int(fp8.quantize(np.array([x]), scale, fp8.E4M3)[0])
    # whatever fp32 gives, the oracle must follow the fp32 product, not the exact one
    assert code == int(fp8.encode(np.array([prod32]), fp8.E4M3)[0])
    if Fraction(float(prod32)) == Fraction(17, 16) and exact > Fraction(17, 16):
        assert code == 0x38  # tie -> even, whereas single rounding of the exact product gives 0x39


# ------------------------------------------------------------------ bf16
def test_bf16_round_hand_values():
    cases = [
        (1.0, 0x3F80),
        (1.0 + 2.0**-8, 0x3F80),  # tie -> even (1.0)
        (1.0 + 3 * 2.0**-8, 0x3F82),  # tie between 1+2^-7 (odd) and 1+2^-6 (even)
        (1.0 + 2.0**-8 + 2.0**-30, 0x3F81),  # just above the tie: a float32 detour would lose this
        (-2.5, 0xC020),
        (0.0, 0x0000),
        (2.0**-133, 0x0001),  # smallest subnormal
        (2.0**-134, 0x0000),  # tie with zero -> even
        (3.3895313892515355e38, 0x7F7F),  # largest finite
    ]
    for v, bits in cases:
        assert int(bf16.round_from_f64(np.array([v]))[0]) == bits, v


def test_bf16_round_matches_torch_on_float32_inputs():
    rng = np.random.default_rng(3)
    v = (rng.standard_normal(100_000) * np.exp2(rng.integers(-30, 30, 100_000))).astype(np.float32)
    ours = bf16.round_from_f64(v.astype(np.float64))
    lib = torch.from_numpy(v).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(ours, lib)
    assert np.array_equal(bf16.decode(ours), torch.from_numpy(v).to(torch.bfloat16).float().numpy())


@pytest.mark.parametrize("fmt", [fp8.E4M3, fp8.E5M2], ids=lambda f: f.name)
def test_walking_a_large_tensor_in_blocks_changes_no_byte(fmt):
    # encode() and quantize() walk tensors above 2^18 elements block by block; the map is elementwise, so the bytes
    # must equal those of the one-pass rule applied with any other split (here: element by element ranges of a prime size)
    n = (1 << 19) + 12345  # two full blocks and a ragged tail
    rng = np.random.default_rng(7)
    v = (rng.standard_normal(n) * np.exp(rng.uniform(-12, 12, n))).astype(np.float32)
    v[::1001] = 0.0
    v[5::5003] = np.inf
    s = np.float32(3.7)
    got = fp8.quantize(v.reshape(-1, 1), s, fmt)
    assert got.shape == (n, 1) and got.dtype == np.uint8
    with np.errstate(over="ignore"):
        prod = (v * s).astype(np.float32)
    want = np.concatenate([fp8._encode_block(prod[i:i + 99991], fmt) for i in range(0, n, 99991)])
    assert np.array_equal(got.reshape(-1), want)
    assert np.array_equal(fp8.encode(prod, fmt), want)
