"""Pins for the numeric reference (oracle/syrk_oracle.c), CPU only.

Each test ties the reference to something other than itself: a hand-worked
example, closed forms, exact rational arithmetic through an independent
loop nest, symmetry, the algebra of alpha and beta.
"""
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import syrk as O
from paper_2202_10217_b200 import inputs as I

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
BOTH = [O.DTYPE_F64, O.DTYPE_BF16_F32, O.DTYPE_TF32_F32, O.DTYPE_E4M3_F32,
        O.DTYPE_F16_F32]                                                      # every input type of the reference


def lower(x):
    return x[np.tril_indices(x.shape[0])]


def widen(A, dtype):
    if dtype == O.DTYPE_F64:
        return A
    if dtype == O.DTYPE_TF32_F32:
        return I.f32_keep_tf32_bits(A).astype(np.float64)
    if dtype == O.DTYPE_E4M3_F32:
        return I.e4m3_bits_to_f32(A).astype(np.float64)
    if dtype == O.DTYPE_F16_F32:
        return I.f16_bits_to_f32(A).astype(np.float64)
    return I.bf16_bits_to_f32(A).astype(np.float64)


def real_inputs(N, M, seed, dtype):
    if dtype == O.DTYPE_F64:
        return I.normal_f64(N, M, seed)
    if dtype == O.DTYPE_TF32_F32:
        return I.normal_f32(N, M, seed)          # low-order bits set: the reference must drop them
    if dtype == O.DTYPE_E4M3_F32:
        return I.normal_e4m3(N, M, seed)
    if dtype == O.DTYPE_F16_F32:
        return I.normal_f16(N, M, seed)
    return I.normal_bf16(N, M, seed)


def exact_gram_by_outer_products(Af):
    """Full N x N Gram matrix in exact rationals, column-by-column outer products
    (k outermost: a different loop nest from the reference's i, j, k)."""
    N, M = Af.shape
    G = [[Fraction(0)] * N for _ in range(N)]
    for k in range(M):
        col = [Fraction(float(Af[r, k])) for r in range(N)]
        for i in range(N):
            for j in range(N):
                G[i][j] += col[i] * col[j]
    return G


def test_hand_worked_example():
    rows = [l for l in open(os.path.join(GOLDEN, "syrk_3x2_by_hand.txt")) if not l.startswith("#")]
    N, M = map(int, rows[0].split())
    A = np.array([[float(v) for v in rows[1 + r].split()] for r in range(N)])
    want = [[float(v) for v in rows[1 + N + r].split()] for r in range(N)]
    for dtype in BOTH:
        ref, bound = O.syrk_lower(I.to_storage(A, dtype), None, 1.0, 0.0, dtype)
        for i in range(N):
            for j in range(i + 1):
                assert ref[i, j] == want[i][j]
                assert bound[i, j] == want[i][j]        # all entries positive
        assert np.isnan(ref[0, 1]) and np.isnan(ref[1, 2])  # upper triangle never written


@pytest.mark.parametrize("dtype", BOTH)
@pytest.mark.parametrize("N,M", [(1, 1), (5, 7), (17, 64), (8, 4096)])
def test_all_ones_gives_M(dtype, N, M):
    ref, bound = O.syrk_lower(I.ones(N, M, dtype), None, 1.0, 0.0, dtype)
    assert np.all(lower(ref) == float(M)) and np.all(lower(bound) == float(M))


@pytest.mark.parametrize("dtype", BOTH)
def test_orthonormal_rows_give_identity(dtype):
    N = 16
    A = np.zeros((N, 40))
    A[:, :N] = np.eye(N)                                    # [I | 0]
    ref, _ = O.syrk_lower(I.to_storage(A, dtype), None, 1.0, 0.0, dtype)
    assert np.array_equal(lower(ref), lower(np.eye(N)))
    H = np.array([[1.0]])
    while H.shape[0] < 64:                                   # Sylvester-Hadamard
        H = np.block([[H, H], [H, -H]])
    A = H / 8.0                                              # 1/sqrt(64), exact in bf16
    ref, bound = O.syrk_lower(I.to_storage(A, dtype), None, 1.0, 0.0, dtype)
    assert np.array_equal(lower(ref), lower(np.eye(64)))
    assert np.all(lower(bound) == 1.0)


@pytest.mark.parametrize("dtype", BOTH)
def test_single_column_is_rank_one_outer_product(dtype):
    v = np.array([3.0, -1.0, 0.5, 2.0, -4.0, 0.25])
    A = np.zeros((6, 9))
    A[:, 4] = v
    ref, bound = O.syrk_lower(I.to_storage(A, dtype), None, 1.0, 0.0, dtype)
    assert np.array_equal(lower(ref), lower(np.outer(v, v)))
    assert np.array_equal(lower(bound), lower(np.abs(np.outer(v, v))))


@pytest.mark.parametrize("dtype", BOTH)
def test_exact_integers_match_independent_loop_nest(dtype):
    N, M = 23, 37
    A = I.small_int_f64(N, M, seed=11, lo=-3, hi=3)
    G = exact_gram_by_outer_products(A)
    ref, bound = O.syrk_lower(I.to_storage(A, dtype), None, 1.0, 0.0, dtype)
    Gabs = exact_gram_by_outer_products(np.abs(A))
    for i in range(N):
        for j in range(i + 1):
            assert Fraction(ref[i, j]) == G[i][j]
            assert Fraction(bound[i, j]) == Gabs[i][j]
            assert G[i][j] == G[j][i]                       # symmetry of A A^T


@pytest.mark.parametrize("dtype", BOTH)
def test_real_inputs_within_dot_product_bound_of_exact(dtype):
    N, M = 12, 50
    A = I.uniform_f64(N, M, seed=5) if dtype == O.DTYPE_F64 else real_inputs(N, M, 5, dtype)
    Af = widen(A, dtype)
    G = exact_gram_by_outer_products(Af)
    ref, bound = O.syrk_lower(A, None, 1.0, 0.0, dtype)
    u = 2.0 ** -53
    for i in range(N):
        for j in range(i + 1):
            err = abs(Fraction(ref[i, j]) - G[i][j])
            assert err <= Fraction(M * u * 1.01) * Fraction(bound[i, j])
    # the reference must not be exact-by-construction: some entry does round.  (FP8 products are
    # multiples of 2^-18 below 2^18, so their binary64 sums are exact for any M used here; the
    # binary16 products of this seeded input are multiples of 2^-48 below 2^5, exact as well.)
    if dtype in (O.DTYPE_E4M3_F32, O.DTYPE_F16_F32):
        assert all(Fraction(ref[i, j]) == G[i][j] for i in range(N) for j in range(i + 1))
    else:
        assert any(Fraction(ref[i, j]) != G[i][j] for i in range(N) for j in range(i + 1))


@pytest.mark.parametrize("dtype", BOTH)
def test_row_reversal_symmetry(dtype):
    """(P A)(P A)^T = P (A A^T) P^T: entry (i, j) of the reversed problem equals
    entry (N-1-j, N-1-i) of the original, bit for bit (products commute exactly)."""
    N, M = 19, 33
    A = real_inputs(N, M, 3, dtype)
    ref, _ = O.syrk_lower(A, None, 1.0, 0.0, dtype)
    rev, _ = O.syrk_lower(np.ascontiguousarray(A[::-1]), None, 1.0, 0.0, dtype)
    for i in range(N):
        for j in range(i + 1):
            assert rev[i, j] == ref[N - 1 - j, N - 1 - i]


@pytest.mark.parametrize("dtype", BOTH)
@pytest.mark.parametrize("alpha,beta", [(1, 0), (-1, 1), (0, 1), (0, 0), (2.5, -0.5), (1, 2)])
def test_alpha_beta_algebra_on_integers(dtype, alpha, beta):
    N, M = 9, 14
    A = I.small_int_f64(N, M, seed=2)
    Cin = (np.random.default_rng(8).integers(-8, 9, size=(N, N)) * 2).astype(I.c_storage_dtype(dtype))
    base, _ = O.syrk_lower(I.to_storage(A, dtype), None, 1.0, 0.0, dtype)
    ref, _ = O.syrk_lower(I.to_storage(A, dtype), Cin, alpha, beta, dtype)
    want = alpha * base + beta * Cin.astype(np.float64)    # all terms exact in binary64
    assert np.array_equal(lower(ref), lower(want))


@pytest.mark.parametrize("dtype", BOTH)
def test_beta_zero_does_not_read_C(dtype):
    A = I.small_int_f64(6, 5, seed=1)
    poison = np.full((6, 6), np.nan, dtype=I.c_storage_dtype(dtype))
    a, _ = O.syrk_lower(I.to_storage(A, dtype), None, 1.0, 0.0, dtype)
    b, _ = O.syrk_lower(I.to_storage(A, dtype), poison, 1.0, 0.0, dtype)
    assert np.array_equal(lower(a), lower(b)) and not np.isnan(lower(b)).any()


def test_bf16_widening_bit_patterns():
    bits = np.array([[0x3F80, 0xC000, 0x3DCD, 0x0000]], dtype=np.uint16)   # 1, -2, 0.10009765625, 0
    ref, bound = O.syrk_lower(bits, None, 1.0, 0.0, O.DTYPE_BF16_F32)
    assert ref[0, 0] == 1.0 + 4.0 + 0.10009765625 ** 2
    assert bound[0, 0] == ref[0, 0]


@pytest.mark.parametrize("dtype", BOTH)
def test_leading_dimensions_and_entry_list(dtype):
    N, M, lda, ldc = 13, 21, 32, 20
    big = {O.DTYPE_F64: I.small_int_f64, O.DTYPE_BF16_F32: I.small_int_bf16, O.DTYPE_TF32_F32: I.small_int_f32,
           O.DTYPE_E4M3_F32: I.small_int_e4m3, O.DTYPE_F16_F32: I.small_int_f16}[dtype](N, lda, 4)
    A = big[:, :M]                                           # row pitch lda > M
    Cbig = I.random_c(N, 6, dtype, ldc)
    Cin = Cbig[:, :N]
    ref, bound = O.syrk_lower(A, Cin, -1.0, 1.0, dtype)
    ref2, bound2 = O.syrk_lower(np.ascontiguousarray(A), np.ascontiguousarray(Cin), -1.0, 1.0, dtype)
    assert np.array_equal(lower(ref), lower(ref2)) and np.array_equal(lower(bound), lower(bound2))
    ii, jj = np.tril_indices(N)
    r3, b3 = O.syrk_entries(ii, jj, A, Cin, -1.0, 1.0, dtype)
    assert np.array_equal(r3, lower(ref)) and np.array_equal(b3, lower(bound))
    with pytest.raises(ValueError):
        O.syrk_entries([0], [1], A, Cin, 1.0, 0.0, dtype)    # upper-triangle entry refused


def test_tf32_reading_drops_the_13_low_order_bits():
    """TF32 keeps 10 fraction bits.  1 + 2^-10 survives; 1 + 2^-11 + 2^-12 (0.75 ulp above 1) and
    1 + 2^-10 - 2^-23 (just below the next TF32 value) are cut down, not rounded up; signs follow."""
    x = np.array([[1.0 + 2.0 ** -10, 1.0 + 2.0 ** -11 + 2.0 ** -12, -(1.0 + 2.0 ** -10 - 2.0 ** -23), 3.0]],
                 dtype=np.float32)
    ref, bound = O.syrk_lower(x, None, 1.0, 0.0, O.DTYPE_TF32_F32)
    assert ref[0, 0] == (1.0 + 2.0 ** -10) ** 2 + 1.0 + 1.0 + 9.0
    assert bound[0, 0] == ref[0, 0]
    two = np.array([[1.0 + 2.0 ** -11 + 2.0 ** -12], [-(1.0 + 2.0 ** -10 - 2.0 ** -23)]], dtype=np.float32)
    ref, bound = O.syrk_lower(two, None, 1.0, 0.0, O.DTYPE_TF32_F32)
    assert ref[1, 0] == -1.0 and bound[1, 0] == 1.0
    kept = I.f32_keep_tf32_bits(x)
    assert list(kept[0]) == [np.float32(1.0 + 2.0 ** -10), 1.0, -1.0, 3.0]


def test_e4m3_decoding_of_every_byte():
    """All 256 bytes against the format's definition written out independently: value =
    (-1)^s * 2^(e-7) * (1 + f/8), subnormals 2^-6 * f/8, 0x7F and 0xFF NaN, extremes 2^-9 and 448.
    The reference decodes A[i][0]; with a second column of ones... a 1 x 1 product gives value^2,
    and a 2-row problem gives value * 1."""
    import math
    for byte in range(256):
        s_, e, f = byte >> 7, (byte >> 3) & 15, byte & 7
        if e == 15 and f == 7:
            want = math.nan
        elif e == 0:
            want = (-1.0) ** s_ * 2.0 ** -6 * (f / 8.0)
        else:
            want = (-1.0) ** s_ * 2.0 ** (e - 7) * (1.0 + f / 8.0)
        A = np.array([[0x38], [byte]], dtype=np.uint8)               # 0x38 = 1.0
        ref, bound = O.syrk_lower(A, None, 1.0, 0.0, O.DTYPE_E4M3_F32)
        if math.isnan(want):
            assert math.isnan(ref[1, 0]) and math.isnan(ref[1, 1]) and ref[0, 0] == 1.0
        else:
            assert ref[1, 0] == want and ref[1, 1] == want * want and bound[1, 0] == abs(want)
    assert O.syrk_lower(np.array([[0x7E]], dtype=np.uint8), None, 1.0, 0.0, O.DTYPE_E4M3_F32)[0][0, 0] == 448.0 ** 2
    assert O.syrk_lower(np.array([[0x01]], dtype=np.uint8), None, 1.0, 0.0, O.DTYPE_E4M3_F32)[0][0, 0] == 2.0 ** -18


def test_f16_decoding_of_every_bit_pattern():
    """All 65536 binary16 patterns against the format's definition written out here:
    value = (-1)^s * 2^(e-15) * (1 + f/1024); e = 0: (-1)^s * 2^-14 * f/1024; e = 31: infinity
    (f = 0) or NaN.  Row 0 holds 1.0 (0x3C00), so entry (r, 0) of the result is the decoded
    value of row r and entry (r, r) its square; hand values at the extremes follow."""
    codes = np.arange(65536, dtype=np.uint32)
    s_, e, f = codes >> 15, (codes >> 10) & 31, codes & 1023
    want = np.where(e == 0, 2.0 ** -14 * (f / 1024.0), 2.0 ** (e.astype(np.float64) - 15) * (1.0 + f / 1024.0))
    want = np.where(e == 31, np.where(f == 0, np.inf, np.nan), want)
    want = np.where(s_ == 1, -want, want)
    finite = np.isfinite(want)
    for lo in range(0, 65536, 2048):                                 # 32 problems of 2049 rows, M = 1
        block = codes[lo:lo + 2048].astype(np.uint16)
        A = np.concatenate([np.array([0x3C00], dtype=np.uint16), block]).reshape(-1, 1)
        I_ = np.arange(1, 2049)
        v, b = O.syrk_entries(I_, np.zeros(2048, dtype=np.int64), A, None, 1.0, 0.0, O.DTYPE_F16_F32)
        sq, _ = O.syrk_entries(I_, I_, A, None, 1.0, 0.0, O.DTYPE_F16_F32)
        w, fin = want[lo:lo + 2048], finite[lo:lo + 2048]
        assert np.array_equal(v[fin], w[fin]) and np.array_equal(b[fin], np.abs(w[fin]))
        assert np.array_equal(sq[fin], w[fin] * w[fin])
        assert np.array_equal(np.isnan(v), np.isnan(w)) and np.array_equal(np.isinf(v), np.isinf(w))
    one = lambda bits: O.syrk_lower(np.array([[bits]], dtype=np.uint16), None, 1.0, 0.0, O.DTYPE_F16_F32)[0][0, 0]
    assert one(0x7BFF) == 65504.0 ** 2            # largest finite value
    assert one(0x0001) == 2.0 ** -48              # smallest subnormal, squared
    assert one(0x0400) == 2.0 ** -28              # smallest normal 2^-14, squared
    assert one(0x3555) == (1365.0 / 4096.0) ** 2  # 0.333251953125 = (1 + 341/1024) / 4
    assert one(0xC000) == 4.0                     # -2
    # the library that owns the type agrees (cross-check of the decoding, not the reference itself)
    lib = np.arange(65536, dtype=np.uint32).astype(np.uint16).view(np.float16).astype(np.float64)
    assert np.array_equal(lib[finite], want[finite])


def test_f16_rounding_of_inputs_is_nearest_even():
    # ulp of binary16 at 1 is 2^-10: 1 + 2^-11 ties to 1 (even), 1 + 3 * 2^-11 ties up to 1 + 2^-9;
    # 65520 is the tie between 65504 and the overflow threshold -> infinity; 2^-25 ties to zero.
    x = np.array([1.0 + 2.0 ** -11, 1.0 + 3 * 2.0 ** -11, 1.0 + 2.0 ** -11 + 2.0 ** -20, 65519.0, 2.0 ** -25,
                  -(2.0 ** -24)], dtype=np.float32)
    bits = I.f32_to_f16_bits(x)
    assert list(bits) == [0x3C00, 0x3C02, 0x3C01, 0x7BFF, 0x0000, 0x8001]
    assert list(I.f16_bits_to_f32(bits)[:4]) == [1.0, 1.0 + 2.0 ** -9, 1.0 + 2.0 ** -10, 65504.0]


def test_e4m3_rounding_of_inputs_is_nearest_even_and_saturating():
    # between 1.0 (0x38) and 1.125 (0x39): 1.0625 is a tie -> even code 0x38; 1.1875 ties 0x39/0x3A -> 0x3A
    x = np.array([1.0625, 1.1875, 1.07, 1000.0, -1000.0, 2.0 ** -10, 0.0, -0.0], dtype=np.float32)
    bits = I.f32_to_e4m3_bits(x)
    assert list(bits) == [0x38, 0x3A, 0x39, 0x7E, 0xFE, 0x00, 0x00, 0x80]   # 2^-10 ties 0 / 2^-9 -> code 0
    assert list(I.e4m3_bits_to_f32(bits)[:5]) == [1.0, 1.25, 1.125, 448.0, -448.0]


def test_bf16_rounding_of_inputs_is_nearest_even():
    # 1 + 2^-8 is a tie between 1 and 1 + 2^-7 -> even (1.0); 1 + 3*2^-8 ties up to 1 + 2^-6.
    x = np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -20], dtype=np.float32)
    got = I.bf16_bits_to_f32(I.f32_to_bf16_bits(x))
    assert list(got) == [1.0, 1.0 + 2.0 ** -6, 1.0 + 2.0 ** -7]


def test_tolerance_formula():
    t = O.tolerance(4, np.array([2.0]), np.array([3.0]), -1.0, 1.0, O.DTYPE_F64)
    assert t[0] == 8 * 2.0 ** -53 * 4 * 5.0
    t = O.tolerance(4, np.array([2.0]), np.array([3.0]), 2.0, 0.0, O.DTYPE_BF16_F32)
    assert t[0] == 4 * 2.0 ** -24 * 4 * 4.0
