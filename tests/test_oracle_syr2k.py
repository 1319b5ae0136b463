"""Pins for the rank-2k reference (oracle/syr2k_oracle.c), CPU only: each test ties it to something
other than itself - the pinned SYRK reference, exact rationals through another loop nest, closed
forms, the exchange symmetry, the algebra of alpha and beta."""
from fractions import Fraction

import numpy as np
import pytest

from oracle import syr2k as R
from oracle import syrk as O
from paper_2202_10217_b200 import inputs as I


def lower(x):
    return x[np.tril_indices(x.shape[0])]


def test_hand_worked_example():
    import os
    rows = [l for l in open(os.path.join(os.path.dirname(__file__), "golden", "syr2k_3x2_by_hand.txt")) if not l.startswith("#")]
    N, M = map(int, rows[0].split())
    A = np.array([[float(v) for v in rows[1 + r].split()] for r in range(N)])
    B = np.array([[float(v) for v in rows[1 + N + r].split()] for r in range(N)])
    want = [[float(v) for v in rows[1 + 2 * N + r].split()] for r in range(N)]
    ref, bound = R.syr2k_lower(A, B, None, 1.0, 0.0)
    for i in range(N):
        for j in range(i + 1):
            assert ref[i, j] == want[i][j]
    assert bound[2, 0] == 5 + 0 + 2 + 2 and bound[2, 2] == 2 * (10 + 6)      # the bound sums absolute products
    ref, _ = R.syr2k_lower(A, B, np.ones((N, N)), 2.0, -3.0)                 # alpha = 2, beta = -3 on C = ones
    assert ref[2, 1] == 2.0 * 8 - 3.0


def test_b_equal_a_is_twice_the_syrk_reference():
    A = I.small_int_f64(23, 31, seed=1)                       # integers: every sum exact
    ref2, bd2 = R.syr2k_lower(A, A.copy(), None, 1.0, 0.0)
    ref1, bd1 = O.syrk_lower(A, None, 1.0, 0.0, O.DTYPE_F64)
    assert np.array_equal(lower(ref2), 2.0 * lower(ref1)) and np.array_equal(lower(bd2), 2.0 * lower(bd1))
    A = I.normal_f64(17, 40, seed=2)                          # reals: a*a + a*a = 2 a*a exactly, so still equal
    ref2, _ = R.syr2k_lower(A, A.copy(), None, 1.0, 0.0)
    ref1, _ = O.syrk_lower(A, None, 1.0, 0.0, O.DTYPE_F64)
    assert np.array_equal(lower(ref2), 2.0 * lower(ref1))


def test_exact_rationals_by_outer_products():
    """Full N x N matrix A B^T + B A^T in exact rationals, k outermost (another loop nest)."""
    N, M = 9, 14
    A, B = I.normal_f64(N, M, seed=3), I.normal_f64(N, M, seed=4)
    G = [[Fraction(0)] * N for _ in range(N)]
    for k in range(M):
        a = [Fraction(float(A[r, k])) for r in range(N)]
        b = [Fraction(float(B[r, k])) for r in range(N)]
        for i in range(N):
            for j in range(N):
                G[i][j] += a[i] * b[j] + b[i] * a[j]
    ref, bound = R.syr2k_lower(A, B, None, 1.0, 0.0)
    u = 2.0 ** -53
    assert all(G[i][j] == G[j][i] for i in range(N) for j in range(N))          # the result is symmetric
    for i in range(N):
        for j in range(i + 1):
            assert abs(Fraction(ref[i, j]) - G[i][j]) <= Fraction(2 * M * u * 1.01) * Fraction(bound[i, j])
    assert any(Fraction(ref[i, j]) != G[i][j] for i in range(N) for j in range(i + 1))   # it does round
    Ai, Bi = I.small_int_f64(N, M, seed=5), I.small_int_f64(N, M, seed=6)
    ref, _ = R.syr2k_lower(Ai, Bi, None, 1.0, 0.0)
    full = Ai @ Bi.T + Bi @ Ai.T                                                   # exact on small integers
    assert np.array_equal(lower(ref), lower(full))


def test_closed_forms():
    N, M = 12, 20
    ones = np.ones((N, M))
    ref, bound = R.syr2k_lower(ones, ones, None, 1.0, 0.0)
    assert np.all(lower(ref) == 2.0 * M) and np.all(lower(bound) == 2.0 * M)
    ref, bound = R.syr2k_lower(I.normal_f64(N, M, seed=7), np.zeros((N, M)), None, 1.0, 0.0)
    assert np.all(lower(ref) == 0.0) and np.all(lower(bound) == 0.0)
    # A = e_p e_q^T (one non-zero), B arbitrary: A B^T + B A^T has row p and column p only
    A = np.zeros((N, M)); A[3, 5] = 2.0
    B = I.small_int_f64(N, M, seed=8)
    ref, _ = R.syr2k_lower(A, B, None, 1.0, 0.0)
    want = np.zeros((N, N)); want[3, :] += 2.0 * B[:, 5]; want[:, 3] += 2.0 * B[:, 5]
    assert np.array_equal(lower(ref), lower(want))
    assert np.isnan(ref[0, 1]) and np.isnan(bound[2, 9])                          # upper triangle never written


def test_exchanging_a_and_b_changes_no_bit():
    A, B = I.normal_f64(15, 33, seed=9), I.normal_f64(15, 33, seed=10)
    r1, b1 = R.syr2k_lower(A, B, None, 1.0, 0.0)
    r2, b2 = R.syr2k_lower(B, A, None, 1.0, 0.0)
    assert np.array_equal(lower(r1), lower(r2)) and np.array_equal(lower(b1), lower(b2))


@pytest.mark.parametrize("alpha,beta", [(1.0, 0.0), (-1.0, 1.0), (0.0, 1.0), (0.0, 0.0), (2.5, -0.5)])
def test_alpha_beta_algebra_on_integers(alpha, beta):
    N, M = 14, 18
    A, B = I.small_int_f64(N, M, seed=11), I.small_int_f64(N, M, seed=12)
    Cin = np.round(I.random_c(N, 13, O.DTYPE_F64) * 4)
    ref, _ = R.syr2k_lower(A, B, Cin, alpha, beta)
    want = alpha * (A @ B.T + B @ A.T) + beta * Cin
    assert np.array_equal(lower(ref), lower(want))
    poisoned = np.full((N, N), np.nan)
    ref0, _ = R.syr2k_lower(A, B, poisoned, alpha, 0.0)                           # beta = 0: C is not read
    assert not np.isnan(lower(ref0)).any()


def test_pitches():
    N, M = 11, 13
    bigA, bigB = I.small_int_f64(N, 20, seed=14), I.small_int_f64(N, 24, seed=15)
    A, B = bigA[:, :M], bigB[:, :M]
    r1, _ = R.syr2k_lower(A, B, None, 1.0, 0.0)
    r2, _ = R.syr2k_lower(np.ascontiguousarray(A), np.ascontiguousarray(B), None, 1.0, 0.0)
    assert np.array_equal(lower(r1), lower(r2))


def test_typed_reference_decodes_through_the_pinned_decoder_and_reduces_to_the_rank_k_reference():
    """Operands in a storage type are decoded by the rank-k reference's decoder (pinned pattern by pattern in
    test_oracle_syrk.py) and then go through the binary64 definition.  Pins: the decoder's output squared is
    the rank-k reference of a one-column problem, bit for bit, for every 8-bit pattern and for sampled 16-bit
    patterns; B = A gives twice the rank-k reference of the same type, bit for bit (all sums are of exactly
    representable products, doubling is exact); the exchange of A and B changes no bit."""
    from oracle import syrk as O
    from paper_2202_10217_b200 import inputs as I
    allbytes = np.arange(256, dtype=np.uint8).reshape(256, 1)
    w = O.widen(allbytes, O.DTYPE_E4M3_F32)
    ref, _ = O.syrk_lower(allbytes, None, 1.0, 0.0, O.DTYPE_E4M3_F32)
    d = np.diag(ref)
    ok = ~np.isnan(w[:, 0])
    assert np.array_equal(d[ok], (w[:, 0] ** 2)[ok]) and np.isnan(d[~ok]).all() and (~ok).sum() == 2
    for dtype in (O.DTYPE_BF16_F32, O.DTYPE_F16_F32):
        pats = np.random.default_rng(5).integers(0, 1 << 16, size=(400, 1)).astype(np.uint16)
        w = O.widen(pats, dtype)[:, 0]
        d = np.diag(O.syrk_lower(pats, None, 1.0, 0.0, dtype)[0])
        fin = np.isfinite(w)
        assert np.array_equal(d[fin], (w ** 2)[fin])
    x = np.array([[1.0 + 2.0 ** -10, 1.0 + 2.0 ** -11 + 2.0 ** -12]], dtype=np.float32)      # TF32 keeps 10 fraction bits
    assert np.array_equal(O.widen(x, O.DTYPE_TF32_F32), np.array([[1.0 + 2.0 ** -10, 1.0]]))
    N, M = 37, 29
    for dtype, gen in ((O.DTYPE_BF16_F32, I.normal_bf16), (O.DTYPE_F16_F32, I.normal_f16), (O.DTYPE_TF32_F32, I.normal_f32),
                       (O.DTYPE_E4M3_F32, I.normal_e4m3)):
        A, Bm = gen(N, M, 3), gen(N, M, 4)
        Cin = I.random_c(N, 5, dtype)
        il = np.tril_indices(N)
        twice, _ = R.syr2k_lower_typed(A, A, None, 1.0, 0.0, dtype)
        once, _ = O.syrk_lower(A, None, 1.0, 0.0, dtype)
        assert np.array_equal(twice[il], 2.0 * once[il])
        ab, bd1 = R.syr2k_lower_typed(A, Bm, Cin, 0.5, -1.0, dtype)
        ba, bd2 = R.syr2k_lower_typed(Bm, A, Cin, 0.5, -1.0, dtype)
        assert np.array_equal(ab[il], ba[il]) and np.array_equal(bd1[il], bd2[il])
        # against exact rational arithmetic on the decoded values (a k-outermost loop nest of its own)
        from fractions import Fraction
        A64, B64 = O.widen(A, dtype), O.widen(Bm, dtype)
        for (i, j) in [(0, 0), (5, 2), (36, 35), (20, 20)]:
            s = Fraction(0)
            for k in range(M):
                s += Fraction(float(A64[i, k])) * Fraction(float(B64[j, k])) + Fraction(float(B64[i, k])) * Fraction(float(A64[j, k]))
            exact = Fraction(0.5) * s - Fraction(float(Cin[i, j]))
            assert abs(Fraction(float(ab[i, j])) - exact) <= Fraction(2 * M * 2.0 ** -53) * Fraction(float(bd1[i, j]) + abs(float(Cin[i, j])))
