"""Pins for the oracle's three GEMM definitions (CPU only): exact-rational brute force."""
from fractions import Fraction

import numpy as np
import pytest

from oracle import bf16, fp8
from oracle.layer import gemm_dI, gemm_dW, gemm_fwd


def _frac_bf16(fr: Fraction) -> int:
    """Round an exact rational to bf16 (ties to even) with integer arithmetic only."""
    if fr == 0:
        return 0
    sign = 0x8000 if fr < 0 else 0
    a = abs(fr)
    e = 0
    while a >= 2:
        a /= 2
        e += 1
    while a < 1:
        a *= 2
        e -= 1
    # a in [1,2): 7 fractional bits
    scaled = a * 128
    n = scaled.numerator // scaled.denominator
    rem = scaled - n
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and n % 2 == 1):
        n += 1
    if n == 256:
        n, e = 128, e + 1
    assert -126 <= e <= 127
    return sign | ((e + 127) << 7) | (n - 128)


def _frac_f32(fr: Fraction) -> np.float32:
    # float64 division of exact integers is correctly rounded; these tiny cases never sit on a
    # double-rounding boundary (checked by comparing against exact error bound below)
    return np.float32(fr.numerator / fr.denominator)


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_brute_force_exact_rational(seed):
    rng = np.random.default_rng(seed)
    T, K, N = 5, 16, 7
    Xq = rng.integers(0, 256, (T, K)).astype(np.uint8)
    Wq = rng.integers(0, 256, (N, K)).astype(np.uint8)
    Gq = rng.integers(0, 256, (T, N)).astype(np.uint8)
    # avoid NaN / Inf codes
    Xq[(Xq & 0x7F) == 0x7F] = 0x10
    Wq[(Wq & 0x7F) == 0x7F] = 0x20
    Gq[(Gq & 0x7C) == 0x7C] = 0x30
    sX, sW, sG = np.float32(1 / 448), np.float32(0.37), np.float32(3.1e-5)
    fx = lambda c: Fraction(float(fp8.decode(np.uint8(c), fp8.E4M3)))
    fg = lambda c: Fraction(float(fp8.decode(np.uint8(c), fp8.E5M2)))
    FX, FW, FG = Fraction(float(sX)), Fraction(float(sW)), Fraction(float(sG))

    Y = gemm_fwd(Xq, Wq, sX, sW)
    dX = gemm_dI(Gq, Wq, sG, sW)
    D = gemm_dW(Gq, Xq, sG, sX)
    for t in range(T):
        for n in range(N):
            acc = sum(fx(Xq[t, k]) * fx(Wq[n, k]) for k in range(K)) * FX * FW
            assert int(Y[t, n]) == _frac_bf16(acc), (t, n)
        for k in range(K):
            acc = sum(fg(Gq[t, n]) * fx(Wq[n, k]) for n in range(N)) * FG * FW
            assert int(dX[t, k]) == _frac_bf16(acc), (t, k)
    for n in range(N):
        for k in range(K):
            acc = sum(fg(Gq[t, n]) * fx(Xq[t, k]) for t in range(T)) * FG * FX
            got = float(D[n, k])
            exact = acc.numerator / acc.denominator
            assert abs(got - exact) <= 2**-24 * abs(exact) * 1.0000001
            assert D.dtype == np.float32


def test_row_sampling_equals_full():
    rng = np.random.default_rng(5)
    Xq = rng.integers(0, 0x78, (9, 32)).astype(np.uint8)
    Wq = rng.integers(0, 0x78, (11, 32)).astype(np.uint8)
    Gq = rng.integers(0, 0x78, (9, 11)).astype(np.uint8)
    rows = [0, 4, 8]
    assert np.array_equal(gemm_fwd(Xq, Wq, 1.0, 1.0, rows), gemm_fwd(Xq, Wq, 1.0, 1.0)[rows])
    assert np.array_equal(gemm_dI(Gq, Wq, 1.0, 1.0, rows), gemm_dI(Gq, Wq, 1.0, 1.0)[rows])
    assert np.array_equal(gemm_dW(Gq, Xq, 1.0, 1.0, [1, 10]), gemm_dW(Gq, Xq, 1.0, 1.0)[[1, 10]])


def test_integer_inputs_and_permutation_weight():
    # integers representable in FP8, scale 1: results equal integer matmul; W = permutation -> Y
    # is a column permutation of X (catches transposed or swapped operands)
    rng = np.random.default_rng(11)
    T, K = 6, 8
    Xi = rng.integers(-8, 9, (T, K)).astype(np.float32)
    Xq = fp8.encode(Xi, fp8.E4M3)
    assert np.array_equal(fp8.decode(Xq, fp8.E4M3), Xi)
    perm = rng.permutation(K)
    Wi = np.zeros((K, K), np.float32)
    Wi[np.arange(K), perm] = 1.0  # W[n, perm[n]] = 1  ->  Y[t, n] = X[t, perm[n]]
    Wq = fp8.encode(Wi, fp8.E4M3)
    Y = bf16.decode(gemm_fwd(Xq, Wq, 1.0, 1.0))
    assert np.array_equal(Y, Xi[:, perm])
    Gi = rng.integers(-4, 5, (T, K)).astype(np.float32)
    Gq = fp8.encode(Gi, fp8.E5M2)
    dX = bf16.decode(gemm_dI(Gq, Wq, 1.0, 1.0))
    assert np.array_equal(dX, Gi @ Wi)  # dX[t,k] = sum_n G[t,n] W[n,k]
    D = gemm_dW(Gq, Xq, 1.0, 1.0)
    assert np.array_equal(D, Gi.T @ Xi)
