"""GPU parity of the Large Block Cholesky driver against the CPU reference (Algorithm 2).

Bar: backward error  |A - L L^T|_ij <= 4 (N+1) 2^-53 (|L||L|^T)_ij  for every i >= j (the
classical bound of a Cholesky factor, which holds whatever the condition number because every
solve is a substitution), and entries of L close to the reference factor for well-conditioned
matrices; matrices whose factorisation is exact in binary64 must match bit for bit; the strict
upper triangle is never touched.
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
    for N, block in ((100, 0), (300, 128)):   # across inner blocks, leaves and panels: substitutions and
        L0 = np.tril(rng.integers(-1, 2, size=(N, N))).astype(np.float64)      # products of small integers
        L0[np.diag_indices(N)] = 16.0                                # and of multiples of 1/16 stay exact
        L, info = factor_on_gpu(L0 @ L0.T, block)
        assert info == 0 and np.array_equal(np.tril(L), L0)


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


@pytest.mark.parametrize("N,block,decades", [(512, 128, 10), (1000, 256, 12), (384, 128, 8)])
def test_ill_conditioned_matrices_keep_the_backward_error_bound(N, block, decades):
    """A = Q diag(d) Q^T with d spread evenly over `decades` powers of ten (condition number 1e8 .. 1e12,
    of the matrix and of the diagonal blocks the panels see): the factor's backward error must stay within
    the classical bound, as the reference's does - a solve through explicit inverses of the diagonal blocks
    would lose it by orders of magnitude here."""
    rng = np.random.default_rng(N)
    Q, _ = np.linalg.qr(rng.standard_normal((N, N)))
    d = np.logspace(0.0, -float(decades), N)
    A = (Q * d) @ Q.T
    A = (A + A.T) / 2
    Lref, info_ref = K.cholesky_lower(A)
    assert info_ref == 0 and K.residual_ok(A, Lref)[0]
    L, info = factor_on_gpu(A, block)
    assert info == 0
    ok, worst = K.residual_ok(A, L)
    assert ok, "worst residual / bound = %g" % worst


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


def test_n32768_leading_columns_against_reference_and_sampled_residual():
    """The benchmark's factorisation (N = 32768, n I + G G^T / 512): the first 256 columns of the factor
    against the reference's leading-columns routine, entry by entry, and the backward-error bound on
    sampled entries of the whole matrix (products of rows of L against the entries of A)."""
    from paper_2202_10217_b200 import inputs as I
    n, c = 32768, 256
    G = torch.from_numpy(I.sweep_factor(n)).cuda()
    A0 = torch.matmul(G, G.T) / float(I.SWEEP_K)                  # input preparation
    A0.diagonal().add_(float(n))
    del G
    panel = A0[:, :c].cpu().numpy()
    A = A0.clone()
    B.cholesky_lower(n, A, n, 0)
    torch.cuda.synchronize()
    assert B.syrk_last_status() == 0 and B.cholesky_last_info() == 0
    Lc_ref, info = K.cholesky_lower_leading(panel)
    assert info == 0
    Lc = A[:, :c].cpu().numpy()
    il = np.tril_indices(n, 0, c)
    assert np.max(np.abs(Lc[il] - Lc_ref[il])) < 1e-11 * np.max(np.abs(Lc_ref[il]))
    iu = np.triu_indices(c, 1)
    assert np.array_equal(Lc[:c][iu], panel[:c][iu])              # strict upper triangle untouched
    gen = torch.Generator(device="cuda").manual_seed(3)
    ii = torch.randint(0, n, (4096,), device="cuda", generator=gen)
    jj = (torch.rand(4096, device="cuda", generator=gen) * (ii + 1).double()).long()
    L = torch.tril(A)
    del A
    got = (L[ii] * L[jj]).sum(dim=1)
    bound = 4.0 * (n + 1) * 2.0 ** -53 * (L[ii].abs() * L[jj].abs()).sum(dim=1)
    assert bool(torch.all((got - A0[ii, jj]).abs() <= bound))
