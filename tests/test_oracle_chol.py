"""Pins for the Cholesky reference (oracle/chol_oracle.c), CPU only."""
import math
import os

import numpy as np

from oracle import chol as K

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def test_hand_worked_example():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "cholesky_3x3_by_hand.txt")) if not l.startswith("#")]
    N = int(rows[0][0])
    A = np.zeros((N, N))
    want = np.zeros((N, N))
    for i in range(N):
        A[i, :i + 1] = [float(v) for v in rows[1 + i]]
        want[i, :i + 1] = [float(v) for v in rows[1 + N + i]]
    A[np.triu_indices(N, 1)] = np.nan                       # the upper triangle must never be read
    L, info = K.cholesky_lower(A)
    assert info == 0
    assert np.array_equal(np.tril(L), want)
    assert np.isnan(L[0, 1]) and np.isnan(L[1, 2])          # ... nor written


def test_pascal_matrix_factor_is_the_binomial_triangle():
    """P_ij = C(i+j, i) is symmetric positive definite with P = L L^T, L_ij = C(i, j):
    every intermediate value is a small integer, so the factorisation is exact."""
    for N in (1, 2, 7, 12):
        P = np.array([[float(math.comb(i + j, i)) for j in range(N)] for i in range(N)])
        L, info = K.cholesky_lower(P)
        want = np.array([[float(math.comb(i, j)) for j in range(N)] for i in range(N)])
        assert info == 0 and np.array_equal(np.tril(L), want)


def test_integer_factor_is_recovered_exactly():
    rng = np.random.default_rng(3)
    N = 40
    L0 = np.tril(rng.integers(-3, 4, size=(N, N))).astype(np.float64)
    L0[np.diag_indices(N)] = rng.integers(1, 5, size=N)     # positive diagonal: the unique factor
    A = L0 @ L0.T                                            # exact in binary64
    L, info = K.cholesky_lower(A)
    assert info == 0 and np.array_equal(np.tril(L), L0)


def test_diagonal_matrix_and_scaling():
    d = np.array([4.0, 9.0, 0.25, 16.0])
    L, info = K.cholesky_lower(np.diag(d))
    assert info == 0 and np.array_equal(np.tril(L), np.diag(np.sqrt(d)))
    rng = np.random.default_rng(1)
    G = rng.standard_normal((30, 30))
    A = G @ G.T + 30 * np.eye(30)
    L1, _ = K.cholesky_lower(A)
    L4, _ = K.cholesky_lower(4.0 * A)                        # chol(4A) = 2 chol(A), exactly (powers of two)
    assert np.array_equal(np.tril(L4), 2.0 * np.tril(L1))


def test_reconstruction_and_library_cross_check():
    rng = np.random.default_rng(7)
    for N in (5, 64, 300):
        G = rng.standard_normal((N, 2 * N))
        A = G @ G.T / N + np.eye(N)
        L, info = K.cholesky_lower(A)
        assert info == 0
        ok, worst = K.residual_ok(A, L)
        assert ok, worst
        ref = np.linalg.cholesky(A)                          # cross-check only
        assert np.allclose(np.tril(L), ref, rtol=1e-11, atol=1e-12)
        assert np.array_equal(np.triu(L, 1), np.triu(A, 1))  # upper triangle untouched
    # a planted mistake (dropping the last update) must break the residual check
    Lbad = L.copy()
    Lbad[N - 1, N - 1] *= 1.0 + 1e-9
    assert not K.residual_ok(A, Lbad)[0]


def test_indefinite_matrix_is_reported():
    A = np.array([[4.0, 2.0, 0.0], [2.0, 1.0, 0.0], [0.0, 0.0, 1.0]])    # second pivot is 1 - 1 = 0
    _, info = K.cholesky_lower(A)
    assert info == 2
    _, info = K.cholesky_lower(np.array([[-1.0]]))
    assert info == 1


def test_leading_columns_routine_equals_the_full_factorisation_bit_for_bit():
    """The restricted loop performs, for the columns it keeps, the very operations of the full one."""
    rng = np.random.default_rng(11)
    for N in (1, 5, 64, 300):
        G = rng.standard_normal((N, N + 3))
        A = G @ G.T / N + np.eye(N)
        full, info = K.cholesky_lower(A)
        assert info == 0
        for c in sorted({1, min(N, 17), N}):
            panel = A[:, :c].copy()
            panel[np.triu_indices(N, 1, c)] = np.nan               # entries above the diagonal are never read
            Lc, info = K.cholesky_lower_leading(panel)
            assert info == 0
            il = np.tril_indices(N, 0, c)
            assert np.array_equal(Lc[il], full[:, :c][il])
            assert np.isnan(Lc[np.triu_indices(N, 1, c)]).all()  # ... nor written
    # closed form: the first columns of the Pascal matrix's factor are binomial coefficients
    N, c = 12, 5
    P = np.array([[float(math.comb(i + j, i)) for j in range(N)] for i in range(N)])
    Lc, info = K.cholesky_lower_leading(P[:, :c].copy())
    want = np.array([[float(math.comb(i, j)) for j in range(c)] for i in range(N)])
    assert info == 0 and np.array_equal(np.tril(Lc), want)
    # the hand-worked 3 x 3 example, first two columns
    rows = [l.split() for l in open(os.path.join(GOLDEN, "cholesky_3x3_by_hand.txt")) if not l.startswith("#")]
    A3 = np.zeros((3, 3)); W3 = np.zeros((3, 3))
    for i in range(3):
        A3[i, :i + 1] = [float(v) for v in rows[1 + i]]
        W3[i, :i + 1] = [float(v) for v in rows[1 + 3 + i]]
    L2, info = K.cholesky_lower_leading(A3[:, :2].copy())
    assert info == 0 and np.array_equal(np.tril(L2), np.tril(W3[:, :2]))
    # a non-positive pivot inside the kept columns is reported, one beyond them is not looked at
    B3 = np.array([[4.0, 0.0, 0.0], [2.0, 1.0, 0.0], [0.0, 0.0, 1.0]])
    assert K.cholesky_lower_leading(B3[:, :2].copy())[1] == 2
    assert K.cholesky_lower_leading(B3[:, :1].copy())[1] == 0
