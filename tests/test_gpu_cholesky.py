"""GPU parity of the Large Block Cholesky driver against the CPU reference (Algorithm 2).

Bar: backward error  |A - L L^T|_ij <= 4 (N+1) 2^-53 (|L||L|^T)_ij  for every i >= j (the
classical bound of a Cholesky factor, with a factor 4 of slack for the leaf inverses), and
entries of L close to the reference factor; matrices whose factorisation is exact in
binary64 and that fit one 32 x 32 inner block must match bit for bit; the strict upper triangle is never touched.
"""
import math

import numpy as np
import pytest
import torch

from oracle import chol as K
from paper_2202_10217_b200 import binding as B

pytestmark = pytest.mark.gpu


def spd(N, seed, shift=1.0):
    rng = np.random.default_rng(seed)
    G = rng.standard_normal((N, max(N // 2, 4)))
    return G @ G.T / max(N // 2, 4) + shift * np.eye(N)


def factor_on_gpu(A, block=0, lda=None):
    N = A.shape[0]
    lda = N + (N & 1) if lda is None else lda
    host = np.full((N + 2, lda), np.nan)                        # NaN above the diagonal and in the guards
    il = np.tril_indices(N)
    body = host[1:N + 1, :N]
    body[il] = A[il]
    dev = torch.from_numpy(host).cuda()
    ptr = dev.data_ptr() + lda * 8
    B.cholesky_lower(N, ptr, lda, block)
    torch.cuda.synchronize()
    assert B.syrk_last_status() == 0
    out = dev.cpu().numpy()
    mask = np.ones(out.shape, dtype=bool)
    mask[1:N + 1, :N][il] = False
    assert np.isnan(out[mask]).all(), "wrote outside the lower triangle"
    return out[1:N + 1, :N], B.cholesky_last_info()


def test_exact_factorisations_are_bit_exact():
    for N in (1, 5, 12):
        P = np.array([[float(math.comb(i + j, i)) for j in range(N)] for i in range(N)])
        L, info = factor_on_gpu(P)
        assert info == 0
        assert np.array_equal(np.tril(L), np.array([[float(math.comb(i, j)) for j in range(N)] for i in range(N)]))
    rng = np.random.default_rng(3)
    N = 30                       # one 32-block of the leaf is Algorithm 2 itself: exact
    L0 = np.tril(rng.integers(-3, 4, size=(N, N))).astype(np.float64)
    L0[np.diag_indices(N)] = rng.integers(1, 5, size=N)
    L, info = factor_on_gpu(L0 @ L0.T)
    assert info == 0 and np.array_equal(np.tril(L), L0)
    N = 100                      # beyond one block the solves multiply by inverses: tolerance, not equality
    L0 = np.tril(rng.integers(-1, 2, size=(N, N))).astype(np.float64)
    L0[np.diag_indices(N)] = 16.0                                # well conditioned
    L, info = factor_on_gpu(L0 @ L0.T)
    assert info == 0 and K.residual_ok(L0 @ L0.T, L)[0]
    assert np.max(np.abs(np.tril(L) - L0)) < 1e-12


@pytest.mark.parametrize("N,block", [(1, 0), (31, 0), (128, 0), (129, 128), (300, 128), (500, 256), (512, 0),
                                     (640, 512), (1100, 256), (1537, 512), (2500, 512)])
def test_matches_reference_within_backward_error(N, block):
    A = spd(N, seed=N)
    L, info = factor_on_gpu(A, block)
    assert info == 0
    ok, worst = K.residual_ok(A, L)
    assert ok, "worst residual / bound = %g" % worst
    Lref, info_ref = K.cholesky_lower(A)
    assert info_ref == 0
    scale = np.sqrt(np.outer(np.diag(A), np.ones(N)))
    assert np.max(np.abs(np.tril(L) - np.tril(Lref)) / scale) < 1e-11


def test_row_pitch_larger_than_n():
    A = spd(700, seed=5)
    L, info = factor_on_gpu(A, 256, lda=1024)
    assert info == 0 and K.residual_ok(A, L)[0]


def test_indefinite_matrix_reports_the_first_bad_pivot():
    A = spd(400, seed=9)
    A[250, 250] = -5.0                                            # pivot 250 becomes negative
    _, info_ref = K.cholesky_lower(A)
    _, info = factor_on_gpu(A, 128)
    assert info == info_ref == 251


def test_large_matrix_against_reference_and_device_residual():
    N = 4096
    A = spd(N, seed=11, shift=float(N) ** 0.5)
    L, info = factor_on_gpu(A)
    assert info == 0
    Lref, _ = K.cholesky_lower(A)
    assert np.max(np.abs(np.tril(L) - np.tril(Lref))) < 1e-10 * np.max(np.abs(Lref))
    ok, worst = K.residual_ok(A, L)
    assert ok, worst
