"""GPU parity of the Hermitian rank-k update (herk_lower) against the CPU reference (Algorithm 1 over the
complex numbers, second factor conjugated).

Bar, per part (real, imaginary) of every entry of the lower triangle:
    |part_gpu - part_ref| <= 8 * 2^-53 * 2M * (|alpha| * Bound_part + |beta| * |C_in part|)
(each part is a sum of 2M real products); bit for bit on Gaussian-integer inputs, whose sums are exact in any
order; the imaginary part of the diagonal is zero and is not read; the strict upper triangle, the padding of
the rows and the guard rows around C are never written; beta == 0 does not read C.
"""
import numpy as np
import pytest
import torch

from oracle import herk as H
from paper_2202_10217_b200 import binding as B
from paper_2202_10217_b200 import inputs as I

pytestmark = pytest.mark.gpu

GUARD = 2
SENTINEL = complex(-7.25e300, 3.5e-300)


def run_herk(A, alpha, beta, Cin=None, lda=None, ldc=None, a_shift=0, c_shift=0, poison=False, nan_diag=False):
    """One call through the C ABI.  a_shift / c_shift: offsets of the operands in binary64 words (an odd value
    breaks the 16-byte alignment and selects the plain-load kernel).  Returns (got, ref, bound)."""
    N, M = A.shape
    lda = max(M, 1) if lda is None else lda
    ldc = max(N, 1) if ldc is None else ldc
    host_a = np.zeros(max(N, 1) * lda * 2 + a_shift)
    if N and M:
        view = host_a[a_shift:a_shift + N * lda * 2].view(np.complex128).reshape(N, lda)
        view[:, :M] = A
    host_c = np.empty((N + 2 * GUARD) * ldc * 2 + c_shift)
    host_c[:c_shift] = SENTINEL.real
    full = host_c[c_shift:].view(np.complex128).reshape(N + 2 * GUARD, ldc)
    full[:] = SENTINEL
    body = full[GUARD:GUARD + N, :N]
    il = np.tril_indices(N)
    if Cin is not None:
        body[il] = Cin[il]
        if nan_diag:
            body.imag[np.diag_indices(N)] = np.nan
    elif poison:
        body[il] = complex(np.nan, np.nan)
    before = host_c.copy()
    dA = torch.from_numpy(host_a).cuda()
    dC = torch.from_numpy(host_c).cuda()
    a_ptr = dA.data_ptr() + 8 * a_shift
    c_ptr = dC.data_ptr() + 8 * (c_shift + GUARD * ldc * 2)
    B.herk_lower(N, M, a_ptr, lda, c_ptr, ldc, alpha, beta)
    torch.cuda.synchronize()
    assert B.syrk_last_status() == 0
    after = dC.cpu().numpy()
    got_full = after[c_shift:].view(np.complex128).reshape(N + 2 * GUARD, ldc)
    was_full = before[c_shift:].view(np.complex128).reshape(N + 2 * GUARD, ldc)
    untouched = np.ones(got_full.shape, dtype=bool)
    untouched[GUARD:GUARD + N, :N][il] = False
    assert np.array_equal(got_full.view(np.uint64).reshape(N + 2 * GUARD, 2 * ldc)[np.repeat(untouched, 2, axis=1)],
                          was_full.view(np.uint64).reshape(N + 2 * GUARD, 2 * ldc)[np.repeat(untouched, 2, axis=1)])
    assert np.array_equal(after[:c_shift], before[:c_shift])
    ref, bound = H.herk_lower(np.ascontiguousarray(A), Cin, alpha, beta)
    return got_full[GUARD:GUARD + N, :N].copy(), ref, bound


def check(got, ref, bound, M, Cin, alpha, beta, exact=False):
    N = got.shape[0]
    il = np.tril_indices(N)
    g, r = got[il], ref[il]
    assert np.all(np.diag(got).imag == 0.0)
    if exact:
        assert np.array_equal(g, r)
        return
    cin = None if Cin is None else Cin[il]
    tol = H.tolerance(M, bound[il], cin, alpha, beta)
    assert np.all(np.abs(g.real - r.real) <= tol.real)
    assert np.all(np.abs(g.imag - r.imag) <= tol.imag)


SHAPES = [(1, 1), (5, 3), (31, 8), (32, 9), (33, 64), (64, 1), (100, 37), (129, 200), (257, 16), (300, 515),
          (700, 96), (1000, 40)]


@pytest.mark.parametrize("N,M", SHAPES)
def test_gaussian_integers_are_bit_exact(N, M):
    A = I.small_int_c128(N, M, seed=100 + N)
    Cin = np.round(I.random_c128(N, 200 + N) * 8)
    got, ref, bound = run_herk(A, 1.0, 0.0, poison=True)              # beta = 0: NaN-filled C is not read
    check(got, ref, bound, M, None, 1.0, 0.0, exact=True)
    got, ref, bound = run_herk(A, -2.0, 0.5, Cin=Cin, nan_diag=True)
    check(got, ref, bound, M, Cin, -2.0, 0.5, exact=True)


@pytest.mark.parametrize("N,M", [(33, 64), (100, 37), (300, 515), (700, 96), (1500, 500)])
@pytest.mark.parametrize("alpha,beta", [(1.0, 0.0), (-1.0, 1.0), (2.5, -0.5)])
def test_normal_inputs_within_the_bound(N, M, alpha, beta):
    A = I.normal_c128(N, M, seed=300 + N)
    Cin = I.random_c128(N, 400 + N) if beta != 0.0 else None
    got, ref, bound = run_herk(A, alpha, beta, Cin=Cin, poison=(beta == 0.0))
    check(got, ref, bound, M, Cin, alpha, beta)
    il = np.tril_indices(N, -1)
    assert np.any(got[il].imag != 0.0)


def test_imaginary_part_has_the_sign_of_the_definition():
    """Two rows, one column: C[1][0] = A[1][0] conj(A[0][0]); with A = [[1], [i]] that is i, with [[i], [1]] it is -i."""
    got, _, _ = run_herk(np.array([[1.0 + 0j], [1j]]), 1.0, 0.0)
    assert got[1, 0] == 1j and got[0, 0] == 1.0 and got[1, 1] == 1.0
    got, _, _ = run_herk(np.array([[1j], [1.0 + 0j]]), 1.0, 0.0)
    assert got[1, 0] == -1j


@pytest.mark.parametrize("lda_pad,ldc_pad", [(0, 3), (5, 0), (7, 4)])
def test_pitches(lda_pad, ldc_pad):
    N, M = 210, 77
    A = I.small_int_c128(N, M, seed=501)
    Cin = np.round(I.random_c128(N, 502) * 8)
    got, ref, bound = run_herk(A, 1.0, 1.0, Cin=Cin, lda=M + lda_pad, ldc=N + ldc_pad)
    check(got, ref, bound, M, Cin, 1.0, 1.0, exact=True)


@pytest.mark.parametrize("a_shift,c_shift", [(1, 0), (0, 1), (1, 1), (2, 2)])
def test_operands_off_the_16_byte_boundary_take_the_plain_kernel(a_shift, c_shift):
    N, M = 150, 45
    A = I.small_int_c128(N, M, seed=503)
    Cin = np.round(I.random_c128(N, 504) * 8)
    got, ref, bound = run_herk(A, 3.0, -1.0, Cin=Cin, a_shift=a_shift, c_shift=c_shift, nan_diag=True)
    check(got, ref, bound, M, Cin, 3.0, -1.0, exact=True)
    A = I.normal_c128(N, M, seed=505)
    got, ref, bound = run_herk(A, 1.0, 0.0, a_shift=a_shift, c_shift=c_shift, poison=True)
    check(got, ref, bound, M, None, 1.0, 0.0)


@pytest.mark.parametrize("alpha,beta,M", [(0.0, 1.0, 9), (1.0, 1.0, 0), (0.0, 0.0, 9), (0.0, -2.0, 9), (1.5, 3.0, 0), (1.0, 0.0, 0)])
def test_quick_returns(alpha, beta, M):
    N = 70
    A = I.small_int_c128(N, M, seed=506)
    Cin = np.round(I.random_c128(N, 507) * 8)
    if (alpha == 0.0 or M == 0) and beta == 1.0:                        # nothing is touched, the diagonal included
        host = Cin.copy()
        dC = torch.from_numpy(host).cuda()
        dA = torch.zeros(max(N * max(M, 1), 1), dtype=torch.complex128, device="cuda")
        B.herk_lower(N, M, dA, max(M, 1), dC, N, alpha, beta)
        torch.cuda.synchronize()
        assert np.array_equal(dC.cpu().numpy().view(np.uint64), Cin.view(np.uint64))
        return
    got, ref, bound = run_herk(A, alpha, beta, Cin=(Cin if beta != 0.0 else None), poison=(beta == 0.0), nan_diag=(beta != 0.0))
    check(got, ref, bound, M, Cin if beta != 0.0 else None, alpha, beta, exact=True)


def test_argument_validation():
    one = torch.zeros(4, dtype=torch.complex128, device="cuda")
    L = B.lib()
    st = torch.cuda.current_stream().cuda_stream
    assert L.herk_lower(-1, 1, one.data_ptr(), 1, one.data_ptr(), 1, 1.0, 0.0, st) == -2
    assert L.herk_lower(2, 2, one.data_ptr(), 1, one.data_ptr(), 2, 1.0, 0.0, st) == -3     # lda < M
    assert L.herk_lower(2, 2, one.data_ptr(), 2, one.data_ptr(), 1, 1.0, 0.0, st) == -3     # ldc < N
    assert L.herk_lower(2, 2, None, 2, one.data_ptr(), 2, 1.0, 0.0, st) == -1
    assert L.herk_lower(2, 2, one.data_ptr(), 2, None, 2, 1.0, 0.0, st) == -1
    assert L.herk_lower(0, 2, None, 2, None, 1, 1.0, 0.0, st) == 0


def test_larger_problem_on_sampled_entries():
    """4096 x 1024 (several rounds of blocks per SM): sampled entries against the definition evaluated for those
    entries on the host (rows of A gathered, the reference applied to the pair), and the whole diagonal."""
    N, M = 4096, 1024
    A = I.normal_c128(N, M, seed=508)
    dA = torch.from_numpy(A).cuda()
    dC = torch.full((N, N), complex(np.nan, np.nan), dtype=torch.complex128, device="cuda")
    B.herk_lower(N, M, dA, M, dC, N, 1.0, 0.0)
    torch.cuda.synchronize()
    assert B.syrk_last_status() == 0
    C = dC.cpu().numpy()
    assert np.isnan(C[np.triu_indices(N, 1)].real).all()
    assert not np.isnan(C[np.tril_indices(N)].real).any() and not np.isnan(C[np.tril_indices(N)].imag).any()
    rng = np.random.default_rng(509)
    ii = rng.integers(0, N, size=600)
    jj = (rng.random(600) * (ii + 1)).astype(np.int64)
    for i, j in zip(ii, jj):
        pair = np.ascontiguousarray(A[[j, i]])                          # row 1 against row 0: entry (1, 0) of a 2 x 2 problem
        ref, bound = H.herk_lower(pair, None, 1.0, 0.0)
        tol = H.tolerance(M, bound[1, 0], None, 1.0, 0.0)
        assert abs(C[i, j].real - ref[1, 0].real) <= tol.real and abs(C[i, j].imag - ref[1, 0].imag) <= tol.imag
        if i == j:
            assert C[i, j].imag == 0.0
    d = np.einsum("ik,ik->i", A, A.conj()).real
    assert np.all(np.diag(C).imag == 0.0) and np.allclose(np.diag(C).real, d, rtol=1e-12)


@pytest.mark.parametrize("alpha,beta", [(1.0, 0.0), (-1.0, 1.0), (2.5, -0.5)])
def test_launch_forms_agree_bit_for_bit(alpha, beta):
    """One block per item and persistent blocks (whose write-out warps store C: a copy for beta = 0, memory-side
    additions for beta = 1 with the diagonal's imaginary part stored as zero) run the same arithmetic: identical
    bits, both within the bound; a NaN imaginary diagonal in C is never read."""
    for n, (N, M, ldc_pad) in enumerate([(40, 25, 0), (1000, 35, 0), (1300, 20, 3), (2500, 17, 0), (4100, 24, 1)]):
        A = I.normal_c128(N, M, seed=600 + n)
        Cin = I.random_c128(N, 700 + n) if beta != 0.0 else None
        outs = []
        for mode in (B.F64_LAUNCH_PER_ITEM, B.F64_LAUNCH_PERSISTENT):
            try:
                B.syrk_set_f64_launch(mode)
                got, ref, bound = run_herk(A, alpha, beta, Cin=Cin, ldc=N + ldc_pad, poison=(beta == 0.0),
                                           nan_diag=(beta != 0.0))
            finally:
                B.syrk_set_f64_launch(B.F64_LAUNCH_AUTO)
            check(got, ref, bound, M, Cin, alpha, beta)
            outs.append(got)
        il = np.tril_indices(N)
        assert np.array_equal(outs[0][il].view(np.uint64), outs[1][il].view(np.uint64))
