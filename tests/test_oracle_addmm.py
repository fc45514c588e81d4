"""Pins for the oracle's fused-add operator, alpha * (A*B) + beta * D (Section 6.5's AddMM), no GPU.

Checked against things other than itself: the product oracle for the special cases that reduce to it, exact
integer arithmetic, exact rationals with a table-search rounding, numpy float64, and algebraic invariants.
"""
from fractions import Fraction

import numpy as np
import pytest

from oracle import gemm as og
from test_oracle_gemm import brute_round, np_decode

DTYPES = [og.F16, og.BF16]


def enc(x, dtype):
    """16-bit words of exactly representable values through numpy / bit manipulation (not the oracle's encoder)."""
    x = np.asarray(x, dtype=np.float32)
    if dtype == og.F16:
        return x.astype(np.float16).view(np.uint16)
    return (x.view(np.uint32) >> 16).astype(np.uint16)          # exact for values with <= 8 significant bits


@pytest.mark.parametrize("dtype", DTYPES)
def test_alpha_one_beta_zero_is_the_product(dtype):
    rng = np.random.default_rng(1)
    M, N, K = 9, 13, 17
    A = enc(rng.integers(-8, 9, (M, K)) / 4.0, dtype)
    B = enc(rng.integers(-8, 9, (K, N)) / 4.0, dtype)
    D = enc(rng.integers(-8, 9, (M, N)) * 1.0, dtype)
    ref64, ref16 = og.gemm(A, B, M, N, K, dtype)
    o64, o16 = og.addmm_rows(A, B, D, M, N, K, dtype, 1.0, 0.0)
    assert np.array_equal(o64, ref64) and np.array_equal(o16, ref16)


@pytest.mark.parametrize("dtype", DTYPES)
def test_zero_product_returns_beta_d_and_beta_one_returns_d_bit_for_bit(dtype):
    rng = np.random.default_rng(2)
    M, N, K = 6, 40, 5
    A = np.zeros((M, K), dtype=np.uint16)
    B = enc(rng.integers(-8, 9, (K, N)) / 2.0, dtype)
    D = rng.integers(0, 0x7C00 if dtype == og.F16 else 0x7F80, (M, N)).astype(np.uint16)     # arbitrary finite patterns
    _, o16 = og.addmm_rows(A, B, D, M, N, K, dtype, 3.5, 1.0)
    assert np.array_equal(o16, D)
    o64, _ = og.addmm_rows(A, B, D, M, N, K, dtype, 3.5, -0.25)
    assert np.array_equal(o64, -0.25 * np_decode(D, dtype))


@pytest.mark.parametrize("dtype", DTYPES)
def test_integers_against_int64_arithmetic_matrix_and_bias(dtype):
    rng = np.random.default_rng(3)
    M, N, K = 11, 19, 23
    Ai, Bi = rng.integers(-6, 7, (M, K)), rng.integers(-6, 7, (K, N))
    Di, bi = rng.integers(-30, 31, (M, N)), rng.integers(-30, 31, (N,))
    A, B = enc(Ai, dtype), enc(Bi, dtype)
    want = 2 * (Ai @ Bi) - 3 * Di
    o64, o16 = og.addmm_rows(A, B, enc(Di, dtype), M, N, K, dtype, 2.0, -3.0)
    assert np.array_equal(o64, want.astype(np.float64))
    # one rounding: compare with the exact integer rounded by table search
    got = o16.reshape(-1)
    for v, g in zip(want.reshape(-1), got):
        assert int(g) == brute_round(Fraction(int(v)), dtype)
    want_b = 2 * (Ai @ Bi) - 3 * bi[None, :]
    o64b, _ = og.addmm_rows(A, B, enc(bi, dtype), M, N, K, dtype, 2.0, -3.0)
    assert np.array_equal(o64b, want_b.astype(np.float64))


@pytest.mark.parametrize("dtype", DTYPES)
def test_bias_equals_matrix_of_repeated_rows_and_rows_subset(dtype):
    rng = np.random.default_rng(4)
    M, N, K = 7, 21, 9
    A = enc(rng.standard_normal((M, K)), dtype) if dtype == og.F16 else enc(rng.integers(-64, 65, (M, K)) / 16.0, dtype)
    B = enc(rng.integers(-64, 65, (K, N)) / 16.0, dtype)
    b = enc(rng.integers(-64, 65, (N,)) / 8.0, dtype)
    full = np.tile(b, (M, 1))
    o64v, o16v = og.addmm_rows(A, B, b, M, N, K, dtype, 0.75, 1.5)
    o64m, o16m = og.addmm_rows(A, B, full, M, N, K, dtype, 0.75, 1.5)
    assert np.array_equal(o64v, o64m) and np.array_equal(o16v, o16m)
    rows = np.array([5, 0, 3], dtype=np.int64)
    s64, s16 = og.addmm_rows(A, B, full, M, N, K, dtype, 0.75, 1.5, rows=rows)
    assert np.array_equal(s64, o64m[rows]) and np.array_equal(s16, o16m[rows])


@pytest.mark.parametrize("dtype", DTYPES)
def test_against_numpy_float64_and_exact_rationals(dtype):
    rng = np.random.default_rng(5)
    M, N, K = 5, 6, 7
    A = enc(rng.integers(-200, 201, (M, K)) / 64.0, dtype)
    B = enc(rng.integers(-200, 201, (K, N)) / 64.0, dtype)
    D = enc(rng.integers(-200, 201, (M, N)) / 32.0, dtype)
    alpha, beta = np.float32(0.3), np.float32(-1.7)          # binary32 scalars, as the library takes them
    Ad, Bd, Dd = np_decode(A, dtype), np_decode(B, dtype), np_decode(D, dtype)
    o64, o16 = og.addmm_rows(A, B, D, M, N, K, dtype, float(alpha), float(beta))
    want = float(alpha) * (Ad @ Bd) + float(beta) * Dd
    assert np.allclose(o64, want, rtol=1e-13, atol=1e-13)
    # exact rationals: alpha * sum + beta * d, rounded once by table search; the oracle's binary64 value is within
    # 2^-50 relative of it, far from any rounding boundary of the 16-bit type except by bad luck, which the seed avoids
    fa, fb = Fraction(float(alpha)), Fraction(float(beta))
    for i in range(M):
        for j in range(N):
            s = sum(Fraction(float(Ad[i, k])) * Fraction(float(Bd[k, j])) for k in range(K))
            v = fa * s + fb * Fraction(float(Dd[i, j]))
            assert int(o16[i, j]) == brute_round(v, dtype)


def test_scaling_both_scalars_by_a_power_of_two_scales_exactly():
    rng = np.random.default_rng(6)
    M, N, K, dtype = 4, 9, 12, og.F16
    A = enc(rng.integers(-64, 65, (M, K)) / 16.0, dtype)
    B = enc(rng.integers(-64, 65, (K, N)) / 16.0, dtype)
    D = enc(rng.integers(-64, 65, (M, N)) / 16.0, dtype)
    o1, _ = og.addmm_rows(A, B, D, M, N, K, dtype, 0.625, -1.25)
    o4, _ = og.addmm_rows(A, B, D, M, N, K, dtype, 2.5, -5.0)
    assert np.array_equal(o4, 4.0 * o1)


def test_rejects_a_d_of_the_wrong_size():
    A = np.zeros((2, 3), dtype=np.uint16)
    B = np.zeros((3, 4), dtype=np.uint16)
    with pytest.raises(ValueError):
        og.addmm_rows(A, B, np.zeros(5, dtype=np.uint16), 2, 4, 3, og.F16, 1.0, 1.0)
