"""Pins for the CPU oracle of C = A*B (no GPU).

Each test checks ``oracle/gemm_oracle.c`` against something other than itself:
numpy's own 16-bit decoders, exact rational arithmetic, closed forms, library
float64 matmul, and algebraic invariants.
"""
from bisect import bisect_left
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import gemm as og
from paper_2608_10803_b200 import synth

DTYPES = [og.F16, og.BF16]


# ---- independent value tables (numpy's decoders, not the oracle's) ----------

def np_decode(bits: np.ndarray, dtype: int) -> np.ndarray:
    bits = np.asarray(bits, dtype=np.uint16)
    if dtype == og.F16:
        return bits.view(np.float16).astype(np.float64)
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def finite_table(dtype: int):
    """Sorted list of (exact value as Fraction, bits) for every finite non-negative pattern."""
    bits = np.arange(0, 0x8000, dtype=np.uint16)
    vals = np_decode(bits, dtype)
    keep = np.isfinite(vals)
    return [(Fraction(float(v)), int(b)) for v, b in zip(vals[keep], bits[keep])]


_TABLES = {}


def brute_round(x: Fraction, dtype: int) -> int:
    """Round an exact rational to the 16-bit type: nearest, ties to even, by table search."""
    if dtype not in _TABLES:
        t = finite_table(dtype)
        _TABLES[dtype] = ([v for v, _ in t], [b for _, b in t])
    vals, bits = _TABLES[dtype]
    sign = 0x8000 if x < 0 else 0
    a = -x if x < 0 else x
    fbits = 10 if dtype == og.F16 else 7
    inf_bits = 0x7C00 if dtype == og.F16 else 0x7F80
    vmax = vals[-1]
    ulp_top = vals[-1] - vals[-2]
    if a >= vmax + ulp_top / 2:        # at or beyond the midpoint to 2^(emax+1): overflow (tie -> even = inf)
        return sign | inf_bits
    i = bisect_left(vals, a)
    if i < len(vals) and vals[i] == a:
        return sign | bits[i]
    if i >= len(vals):
        return sign | bits[-1]
    lo, hi = vals[i - 1], vals[i]
    if a - lo < hi - a:
        return sign | bits[i - 1]
    if a - lo > hi - a:
        return sign | bits[i]
    return sign | (bits[i - 1] if bits[i - 1] % 2 == 0 else bits[i])


# ---- 16-bit decode / encode --------------------------------------------------

@pytest.mark.parametrize("dtype", DTYPES)
def test_decode_all_patterns_match_numpy(dtype):
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    got = og.decode16(bits, dtype)
    want = np_decode(bits, dtype)
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan], want[~nan])
    assert np.array_equal(np.signbit(got[~nan]), np.signbit(want[~nan]))


@pytest.mark.parametrize("dtype", DTYPES)
def test_encode_roundtrip_all_patterns(dtype):
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    vals = np_decode(bits, dtype)
    ok = ~np.isnan(vals)
    back = og.encode16(vals[ok], dtype)
    assert np.array_equal(back, bits[ok])


@pytest.mark.parametrize("dtype", DTYPES)
def test_encode_midpoints_and_neighbours_vs_exact_rationals(dtype):
    """Every midpoint between adjacent values (the tie cases) and points just off it."""
    t = finite_table(dtype)
    vals = [v for v, _ in t]
    rng = np.random.default_rng(5)
    picks = list(range(0, 40)) + list(range(1000, 1040)) + [len(vals) - 2 - i for i in range(40)]
    picks += [int(i) for i in rng.integers(0, len(vals) - 1, 300)]
    xs = []
    for i in picks:
        lo, hi = vals[i], vals[i + 1]
        mid = (lo + hi) / 2
        eps = (hi - lo) / 1024
        xs += [mid, mid - eps, mid + eps, lo + eps, hi - eps]
    # overflow boundary
    top = vals[-1]
    half_ulp = (vals[-1] - vals[-2]) / 2
    xs += [top + half_ulp, top + half_ulp - half_ulp / 512, top + half_ulp * 3]
    xs += [-x for x in xs]
    xd = np.array([float(x) for x in xs], dtype=np.float64)
    assert all(Fraction(float(d)) == x for d, x in zip(xd, xs)), "test points must be exact doubles"
    got = og.encode16(xd, dtype)
    want = np.array([brute_round(x, dtype) for x in xs], dtype=np.uint16)
    assert np.array_equal(got, want)


def test_encode_f16_matches_numpy_on_random_doubles():
    rng = np.random.default_rng(11)
    x = np.concatenate([rng.normal(0, 1, 20000), rng.normal(0, 3000, 20000),
                        rng.normal(0, 1e-6, 20000), rng.uniform(-7e4, 7e4, 5000)])
    with np.errstate(over="ignore"):
        want = x.astype(np.float16).view(np.uint16)
    assert np.array_equal(og.encode16(x, og.F16), want)


def test_encode_special_values():
    for dtype, inf in [(og.F16, 0x7C00), (og.BF16, 0x7F80)]:
        got = og.encode16(np.array([np.inf, -np.inf, 0.0, -0.0, 1e300, -1e300]), dtype)
        assert list(got) == [inf, inf | 0x8000, 0, 0x8000, inf, inf | 0x8000]
        n = og.encode16(np.array([np.nan]), dtype)[0]
        assert np.isnan(np_decode(np.array([n], dtype=np.uint16), dtype)[0])


# ---- the product --------------------------------------------------------------

def rand_bits(rows, cols, dtype, seed, dist=("uniform", -1.0, 1.0)):
    return synth.bits(synth.draw_operand(rows, cols, dist, seed, dtype))


@pytest.mark.parametrize("dtype", DTYPES)
def test_identity_and_permutation_are_bit_exact(dtype):
    M, K = 37, 53
    A = rand_bits(M, K, dtype, 1)
    one = og.encode16(np.array([1.0]), dtype)[0]
    I = np.zeros((K, K), dtype=np.uint16)
    I[np.arange(K), np.arange(K)] = one
    _, C16 = og.gemm(A, I, M, K, K, dtype)
    assert np.array_equal(C16, A)
    perm = np.random.default_rng(3).permutation(K)
    P = np.zeros((K, K), dtype=np.uint16)
    P[perm, np.arange(K)] = one            # column j of A*P is column perm[j] of A
    _, C16 = og.gemm(A, P, M, K, K, dtype)
    assert np.array_equal(C16, A[:, perm])


@pytest.mark.parametrize("dtype", DTYPES)
def test_rank1_outer_product_closed_form(dtype):
    """K = 1: c_ij = RN16(a_i * b_j); the product of two short significands is exact."""
    M, N = 41, 29
    a = rand_bits(M, 1, dtype, 7)
    b = rand_bits(1, N, dtype, 8)
    C64, C16 = og.gemm(a, b, M, N, 1, dtype)
    av = [Fraction(float(v)) for v in np_decode(a.reshape(-1), dtype)]
    bv = [Fraction(float(v)) for v in np_decode(b.reshape(-1), dtype)]
    for i in range(M):
        for j in range(N):
            exact = av[i] * bv[j]
            assert Fraction(float(C64[i, j])) == exact
            assert int(C16[i, j]) == brute_round(exact, dtype)


@pytest.mark.parametrize("dtype", DTYPES)
def test_integer_inputs_match_integer_arithmetic_bit_exactly(dtype):
    """Entries in [-8, 8]: every partial sum is an exact integer; outputs beyond the
    type's exact-integer range (2048 / 256) exercise the single final rounding."""
    M, N, K = 19, 23, 6000
    A = synth.bits(synth.draw_operand(M, K, ("integer", -8, 8), 21, dtype))
    B = synth.bits(synth.draw_operand(K, N, ("integer", -8, 8), 22, dtype))
    Ai = np_decode(A, dtype).astype(np.int64)
    Bi = np_decode(B, dtype).astype(np.int64)
    Ci = Ai @ Bi
    C64, C16 = og.gemm(A, B, M, N, K, dtype)
    assert np.array_equal(C64, Ci.astype(np.float64))
    want = np.array([[brute_round(Fraction(int(v)), dtype) for v in row] for row in Ci], dtype=np.uint16)
    assert np.array_equal(C16, want)
    limit = 2048 if dtype == og.F16 else 256
    assert (np.abs(Ci) > limit).any(), "case must include outputs that need rounding"


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("shape", [(64, 48, 300), (5, 130, 1), (1, 1, 1000), (33, 7, 129)])
def test_against_numpy_float64_matmul(dtype, shape):
    M, N, K = shape
    A = rand_bits(M, K, dtype, 31)
    B = rand_bits(K, N, dtype, 32, dist=("normal", 0.0, 0.5))
    C64, _ = og.gemm(A, B, M, N, K, dtype)
    Ad, Bd = np_decode(A, dtype), np_decode(B, dtype)
    ref = Ad @ Bd
    bound = K * 2.0 ** -52 * (np.abs(Ad) @ np.abs(Bd)) + 1e-300
    assert np.all(np.abs(C64 - ref) <= bound)
    tref = (torch.from_numpy(Ad) @ torch.from_numpy(Bd)).numpy()
    assert np.all(np.abs(C64 - tref) <= bound)


@pytest.mark.parametrize("dtype", DTYPES)
def test_exact_rational_brute_force_tiny(dtype):
    M, N, K = 6, 7, 8
    A = rand_bits(M, K, dtype, 41)
    B = rand_bits(K, N, dtype, 42)
    C64, C16 = og.gemm(A, B, M, N, K, dtype)
    Ad, Bd = np_decode(A, dtype), np_decode(B, dtype)
    for i in range(M):
        for j in range(N):
            exact = sum(Fraction(float(Ad[i, k])) * Fraction(float(Bd[k, j])) for k in range(K))
            absum = sum(abs(Fraction(float(Ad[i, k])) * Fraction(float(Bd[k, j]))) for k in range(K))
            assert abs(Fraction(float(C64[i, j])) - exact) <= K * Fraction(1, 2 ** 53) * absum
            # the 16-bit result is the rounding of the fp64 sum
            assert int(C16[i, j]) == brute_round(Fraction(float(C64[i, j])), dtype)


def test_transposed_operand_would_be_caught():
    """A non-symmetric case where A*B != A*B^T and != A^T*B: guards an index slip."""
    dtype = og.F16
    n = 16
    A = rand_bits(n, n, dtype, 51)
    B = rand_bits(n, n, dtype, 52)
    C64, _ = og.gemm(A, B, n, n, n, dtype)
    Ad, Bd = np_decode(A, dtype), np_decode(B, dtype)
    assert np.allclose(C64, Ad @ Bd, rtol=0, atol=1e-12)
    assert not np.allclose(C64, Ad @ Bd.T, atol=1e-3)
    assert not np.allclose(C64, Ad.T @ Bd, atol=1e-3)


@pytest.mark.parametrize("dtype", DTYPES)
def test_layout_flags(dtype):
    M, N, K = 21, 34, 55
    A = rand_bits(M, K, dtype, 61)
    B = rand_bits(K, N, dtype, 62)
    C64, C16 = og.gemm(A, B, M, N, K, dtype)
    At = np.ascontiguousarray(A.T)       # column-major storage of A
    Bt = np.ascontiguousarray(B.T)       # column-major storage of B
    for la, lb, a, b in [(og.COL_MAJOR, og.ROW_MAJOR, At, B), (og.ROW_MAJOR, og.COL_MAJOR, A, Bt),
                         (og.COL_MAJOR, og.COL_MAJOR, At, Bt)]:
        D64, D16 = og.gemm(a, b, M, N, K, dtype, la, lb)
        assert np.array_equal(D64, C64) and np.array_equal(D16, C16)


@pytest.mark.parametrize("dtype", DTYPES)
def test_power_of_two_scaling_and_block_concatenation(dtype):
    M, N, K = 24, 40, 96
    A = rand_bits(M, K, dtype, 71)
    B = rand_bits(K, N, dtype, 72)
    C64, _ = og.gemm(A, B, M, N, K, dtype)
    # scaling A by 2^3 is exact in the 16-bit type (values in [-1,1]) and scales C exactly
    A8 = og.encode16(np_decode(A, dtype) * 8.0, dtype).reshape(M, K)
    assert np.array_equal(np_decode(A8, dtype), np_decode(A, dtype) * 8.0)
    D64, _ = og.gemm(A8, B, M, N, K, dtype)
    assert np.array_equal(D64, C64 * 8.0)
    # row blocks and column blocks
    top, _ = og.gemm(A[:10], B, 10, N, K, dtype)
    assert np.array_equal(top, C64[:10])
    left, _ = og.gemm(A, np.ascontiguousarray(B[:, :13]), M, 13, K, dtype)
    assert np.array_equal(left, C64[:, :13])


def test_row_subset_equals_full():
    dtype = og.BF16
    M, N, K = 50, 20, 64
    A = rand_bits(M, K, dtype, 81)
    B = rand_bits(K, N, dtype, 82)
    C64, C16 = og.gemm(A, B, M, N, K, dtype)
    rows = [0, 49, 7, 7, 31]
    S64, S16 = og.gemm_rows(A, B, M, N, K, dtype, rows=rows)
    assert np.array_equal(S64, C64[rows]) and np.array_equal(S16, C16[rows])


def test_degenerate_sizes():
    dtype = og.F16
    A = np.zeros((3, 0), dtype=np.uint16)
    B = np.zeros((0, 4), dtype=np.uint16)
    C64, C16 = og.gemm(A, B, 3, 4, 0, dtype)          # K = 0: all zeros
    assert not C64.any() and not C16.any()
    C64, _ = og.gemm(np.zeros((0, 5), np.uint16), np.zeros((5, 4), np.uint16), 0, 4, 5, dtype)
    assert C64.shape == (0, 4)


def test_rel_fro_error_against_numpy():
    dtype = og.F16
    rng = np.random.default_rng(9)
    ref = rng.normal(0, 3, (30, 30))
    got = og.encode16(ref, dtype)
    err, bad = og.rel_fro_error(got, ref, dtype)
    want = np.linalg.norm(np_decode(got, dtype) - ref) / np.linalg.norm(ref)
    assert bad == 0 and abs(err - want) <= 1e-15
    assert 1e-4 < err < 5e-4       # rounding to fp16 alone: about 0.58 * 2^-11 relative


def test_thread_count_does_not_change_result():
    dtype = og.F16
    M, N, K = 40, 64, 200
    A = rand_bits(M, K, dtype, 91)
    B = rand_bits(K, N, dtype, 92)
    a, _ = og.gemm(A, B, M, N, K, dtype, nthreads=1)
    b, _ = og.gemm(A, B, M, N, K, dtype, nthreads=4)
    assert np.array_equal(a, b)
