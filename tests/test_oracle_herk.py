"""Pins for the Hermitian rank-k reference (oracle/herk_oracle.c), CPU only: each test ties it to something
other than itself - a hand-worked example, the pinned symmetric reference, a library product on Gaussian
integers, closed forms, invariances that fix the sign of the imaginary part and the conjugation."""
import os

import numpy as np
import pytest

from oracle import herk as H
from oracle import syrk as O
from paper_2202_10217_b200 import inputs as I


def lower(x):
    return x[np.tril_indices(x.shape[0])]


def test_hand_worked_example():
    rows = [l for l in open(os.path.join(os.path.dirname(__file__), "golden", "herk_3x2_by_hand.txt")) if not l.startswith("#")]
    N, M = map(int, rows[0].split())

    def pairs(line):
        v = [float(x) for x in line.split()]
        return [complex(v[2 * q], v[2 * q + 1]) for q in range(len(v) // 2)]

    A = np.array([pairs(rows[1 + r]) for r in range(N)], dtype=np.complex128)
    want = [pairs(rows[1 + N + r]) for r in range(N)]
    ref, bound = H.herk_lower(A, None, 1.0, 0.0)
    for i in range(N):
        for j in range(i + 1):
            assert ref[i, j] == want[i][j], (i, j)
    assert bound[1, 0] == complex(3.0, 3.0) and bound[2, 2].real == 10.0      # sums of absolute products, per part
    assert np.isnan(ref[0, 1].real) and np.isnan(bound[0, 2].imag)              # upper triangle never written
    ref, _ = H.herk_lower(A, np.full((N, N), 1.0 + 2.0j), 2.0, -3.0)           # alpha = 2, beta = -3 on C = 1 + 2i
    assert ref[2, 1] == 2.0 * (-4 - 1j) - 3.0 * (1 + 2j)
    assert ref[1, 1] == 2.0 * 3 - 3.0                                          # the diagonal stays real


def test_a_real_matrix_gives_the_symmetric_reference_and_no_imaginary_part():
    Ar = I.normal_f64(19, 37, seed=1)
    ref, bound = H.herk_lower(Ar.astype(np.complex128), None, 1.0, 0.0)
    sym, sym_bound = O.syrk_lower(Ar, None, 1.0, 0.0, O.DTYPE_F64)
    assert np.array_equal(lower(ref).real, lower(sym)) and np.all(lower(ref).imag == 0.0)
    assert np.array_equal(lower(bound).real, lower(sym_bound)) and np.all(lower(bound).imag == 0.0)
    ref, _ = H.herk_lower(1j * Ar.astype(np.complex128), None, 1.0, 0.0)       # (i A)(i A)^H = A A^T
    assert np.array_equal(lower(ref).real, lower(sym)) and np.all(lower(ref).imag == 0.0)


def test_gaussian_integers_against_a_library_product():
    A = I.small_int_c128(21, 29, seed=2)
    ref, bound = H.herk_lower(A, None, 1.0, 0.0)
    full = A @ A.conj().T                                                      # exact on small integers
    assert np.array_equal(lower(ref), lower(full))
    assert np.array_equal(lower(bound).real, lower(np.abs(A.real) @ np.abs(A.real).T + np.abs(A.imag) @ np.abs(A.imag).T))
    assert np.array_equal(lower(bound).imag, lower(np.abs(A.imag) @ np.abs(A.real).T + np.abs(A.real) @ np.abs(A.imag).T))
    assert np.any(lower(ref).imag != 0.0)
    A = I.normal_c128(17, 45, seed=3)                                          # reals: within the stated bound
    ref, bound = H.herk_lower(A, None, 1.0, 0.0)
    full = A @ A.conj().T
    tol = H.tolerance(45, bound, None, 1.0, 0.0)
    assert np.all(np.abs(lower(ref).real - lower(full).real) <= lower(tol).real)
    assert np.all(np.abs(lower(ref).imag - lower(full).imag) <= lower(tol).imag)


def test_rows_with_unit_phases_give_the_identity():
    M = 16
    Hd = np.array([[1.0]])
    while Hd.shape[0] < M:
        Hd = np.block([[Hd, Hd], [Hd, -Hd]])                                   # Sylvester-Hadamard, +-1
    phases = np.array([1j ** p for p in range(M)])
    A = (phases[:, None] * Hd) / 4.0                                           # rows orthonormal, scale exact
    ref, _ = H.herk_lower(A, None, 1.0, 0.0)
    assert np.array_equal(np.tril(np.nan_to_num(ref)), np.eye(M, dtype=np.complex128))
    E = np.zeros((5, 9), dtype=np.complex128)                                  # [D | 0] with unit phases
    for p in range(5):
        E[p, p] = 1j ** (p + 1)
    ref, _ = H.herk_lower(E, None, 1.0, 0.0)
    assert np.array_equal(np.tril(np.nan_to_num(ref)), np.eye(5, dtype=np.complex128))


def test_multiplying_columns_by_i_changes_no_bit():
    A = I.normal_c128(13, 22, seed=4)
    r1, b1 = H.herk_lower(A, None, 1.0, 0.0)
    turned = A.copy()
    turned[:, ::2] = turned[:, ::2] * 1j                                       # exact: (a, b) -> (-b, a)
    assert np.array_equal(turned[:, 0].real, -A[:, 0].imag)
    r2, b2 = H.herk_lower(turned, None, 1.0, 0.0)
    assert np.array_equal(lower(r1), lower(r2)) and np.array_equal(lower(b1), lower(b2))


def test_exchanging_two_rows_gives_the_conjugate():
    A = I.normal_c128(8, 15, seed=5)
    r1, _ = H.herk_lower(A, None, 1.0, 0.0)
    swapped = A.copy()
    swapped[[2, 6]] = swapped[[6, 2]]
    r2, _ = H.herk_lower(swapped, None, 1.0, 0.0)
    assert r2[6, 2] == np.conj(r1[6, 2]) and r2[6, 2].imag != 0.0              # C[2][6] = conj(C[6][2])
    assert r2[6, 6] == r1[2, 2] and r2[2, 2] == r1[6, 6] and r1[6, 6].imag == 0.0
    assert r2[6, 4] == np.conj(r1[4, 2]) and r2[4, 2] == np.conj(r1[6, 4])     # rows between the two


@pytest.mark.parametrize("alpha,beta", [(1.0, 0.0), (-1.0, 1.0), (0.0, 1.0), (0.0, 0.0), (2.5, -0.5)])
def test_alpha_beta_algebra_on_integers(alpha, beta):
    N, M = 14, 18
    A = I.small_int_c128(N, M, seed=6)
    Cin = np.round(I.random_c128(N, 7) * 4)
    clean = Cin.copy()
    clean.imag[np.diag_indices(N)] = 0.0
    Cin.imag[np.diag_indices(N)] = np.nan                                      # imaginary diagonal: never read
    ref, _ = H.herk_lower(A, Cin, alpha, beta)
    want = alpha * (A @ A.conj().T) + beta * clean
    assert np.array_equal(lower(ref), lower(want))
    assert np.all(np.diag(ref).imag == 0.0)
    poisoned = np.full((N, N), complex(np.nan, np.nan))
    ref0, _ = H.herk_lower(A, poisoned, alpha, 0.0)                            # beta = 0: C is not read
    assert not np.isnan(lower(ref0).real).any() and not np.isnan(lower(ref0).imag).any()


def test_pitches():
    N, M = 11, 13
    big = I.small_int_c128(N, 20, seed=8)
    A = big[:, :M]
    r1, _ = H.herk_lower(A, None, 1.0, 0.0)
    r2, _ = H.herk_lower(np.ascontiguousarray(A), None, 1.0, 0.0)
    assert np.array_equal(lower(r1), lower(r2))
    Cbig = np.round(I.random_c128(N, 9, ldc=N + 3) * 4)
    r3, _ = H.herk_lower(A, Cbig[:, :N], 1.0, 1.0)
    r4, _ = H.herk_lower(A, np.ascontiguousarray(Cbig[:, :N]), 1.0, 1.0)
    assert np.array_equal(lower(r3), lower(r4))
