"""GPU parity of syr2k_lower (binary64), through the C ABI, against the CPU reference of the rank-2k
update, entry by entry:  |C_gpu - C_ref| <= 8 * 2^-53 * 2M * (|alpha| Bd + |beta| |C_in|)  with
Bd = |A||B|^T + |B||A|^T (2M products per entry); integer-valued inputs bit for bit.  Everything outside
the lower triangle must stay bitwise untouched."""
import numpy as np
import pytest
import torch

from oracle import syr2k as R
from paper_2202_10217_b200 import binding as B
from paper_2202_10217_b200 import inputs as I

from gpu_util import sentinel_array

pytestmark = pytest.mark.gpu
GUARD = 3


def run(A, Bm, alpha, beta, Cin=None, lda=None, ldb=None, ldc=None, a_off=0, b_off=0, poison=False):
    N, M = A.shape
    lda = max(M, 1) if lda is None else lda
    ldb = max(M, 1) if ldb is None else ldb
    ldc = max(N, 1) if ldc is None else ldc

    def up(X, ld, off):
        buf = torch.zeros(off + max(N, 1) * ld, dtype=torch.float64, device="cuda")
        if N and M:
            buf[off:off + N * ld].view(N, ld)[:, :M].copy_(torch.from_numpy(np.ascontiguousarray(X)))
        return buf, buf.data_ptr() + 8 * off

    ka, pa = up(A, lda, a_off)
    kb, pb = up(Bm, ldb, b_off)
    host_c = sentinel_array((N + 2 * GUARD, ldc), np.float64)
    body = host_c[GUARD:GUARD + N, :N]
    il = np.tril_indices(N)
    if Cin is not None:
        body[il] = Cin[il]
    elif poison:
        body[il] = np.nan
    before = host_c.copy()
    dev_c = torch.from_numpy(host_c).cuda()
    B.syr2k_lower(N, M, pa, lda, pb, ldb, dev_c.data_ptr() + 8 * GUARD * ldc, ldc, alpha, beta)
    torch.cuda.synchronize()
    assert B.syrk_last_status() == 0
    after = dev_c.cpu().numpy()
    mask = np.ones(after.shape, dtype=bool)
    mask[GUARD:GUARD + N, :N][il] = False
    assert np.array_equal(after.view(np.uint64)[mask], before.view(np.uint64)[mask]), "wrote outside the lower triangle"
    got = after[GUARD:GUARD + N, :N]
    ref, bound = R.syr2k_lower(np.ascontiguousarray(A), np.ascontiguousarray(Bm), Cin, alpha, beta if Cin is not None else 0.0)
    return got, ref, bound


def check(got, ref, bound, M, alpha, beta, Cin, exact=False):
    il = np.tril_indices(got.shape[0])
    g, r = got[il], ref[il]
    assert not np.isnan(g).any()
    if exact:
        assert np.array_equal(g, r), "max abs diff %g" % np.max(np.abs(g - r))
        return
    tol = R.tolerance(M, bound[il], None if Cin is None else np.abs(Cin[il]), alpha, beta)
    bad = np.abs(g - r) > tol
    assert not bad.any(), "%d entries out of tolerance" % int(bad.sum())


# below one tile, ragged tiles and K-steps, triangle-block sizes (>= 12 tile rows of 32), large
SIZES = [(1, 1), (5, 3), (31, 17), (32, 16), (33, 50), (100, 64), (257, 130), (512, 256), (1000, 70), (1300, 40),
         (2100, 96)]


def test_real_inputs_within_tolerance():
    for n, (N, M) in enumerate(SIZES):
        A, Bm = I.normal_f64(N, M, 5000 + n), I.normal_f64(N, M, 5100 + n)
        got, ref, bound = run(A, Bm, 1.0, 0.0)
        check(got, ref, bound, M, 1.0, 0.0, None)


def test_integer_inputs_are_bit_exact():
    for n, (N, M) in enumerate(SIZES):
        A, Bm = I.small_int_f64(N, M, 5200 + n), I.small_int_f64(N, M, 5300 + n)
        got, ref, bound = run(A, Bm, 1.0, 0.0)
        check(got, ref, bound, M, 1.0, 0.0, None, exact=True)


@pytest.mark.parametrize("alpha,beta", [(-1.0, 1.0), (0.0, 1.0), (0.0, 0.0), (2.5, -0.5), (1.0, 2.0)])
def test_alpha_beta_pitches_offsets(alpha, beta):
    N, M = 1100, 48
    A, Bm = I.small_int_f64(N, M, 5400), I.small_int_f64(N, M, 5401)
    Cin = I.random_c(N, 5402, I.DTYPE_F64)
    got, ref, bound = run(A, Bm, alpha, beta, Cin, lda=M + 4, ldb=M + 10, ldc=N + 10, a_off=2, b_off=6)
    check(got, ref, bound, M, alpha, beta, Cin)
    got, ref, bound = run(A, Bm, alpha, beta, Cin, ldc=N + 3)                       # odd pitch of C: scalar stores
    check(got, ref, bound, M, alpha, beta, Cin)


def test_nan_poison_unaligned_operands_and_symmetry():
    N, M = 300, 45
    A, Bm = I.normal_f64(N, M, 5500), I.normal_f64(N, M, 5501)
    got, ref, bound = run(A, Bm, 1.0, 0.0, poison=True)                            # beta = 0: C is not read
    check(got, ref, bound, M, 1.0, 0.0, None)
    got2, _, _ = run(Bm, A, 1.0, 0.0)                                               # exchanging A and B
    check(got2, ref, bound, M, 1.0, 0.0, None)
    got3, _, _ = run(A, Bm, 1.0, 0.0, lda=M, a_off=1)                               # odd pitch / base: plain-load kernel
    check(got3, ref, bound, M, 1.0, 0.0, None)
    got4, ref4, bound4 = run(A, A.copy(), 1.0, 0.0)                                 # B = A: twice the rank-k update
    check(got4, ref4, bound4, M, 1.0, 0.0, None)


def test_square_schedule_and_argument_errors():
    N, M = 1056, 96
    A, Bm = I.normal_f64(N, M, 5600), I.normal_f64(N, M, 5601)
    Cin = I.random_c(N, 5602, I.DTYPE_F64)
    try:
        B.syrk_set_schedule(B.SCHEDULE_SQUARE)
        got, ref, bound = run(A, Bm, -1.0, 1.0, Cin)
    finally:
        B.syrk_set_schedule(B.SCHEDULE_DEFAULT)
    check(got, ref, bound, M, -1.0, 1.0, Cin)
    d = torch.zeros(64 * 64, dtype=torch.float64, device="cuda")
    for kwargs, code in [(dict(ldb=15), -3), (dict(lda=15), -3), (dict(Bm=None), -1), (dict(N=-1), -2)]:
        args = dict(N=64, M=16, A=d, lda=16, Bm=d, ldb=16, C=d, ldc=64, alpha=1.0, beta=0.0)
        args.update(kwargs)
        with pytest.raises(B.SyrkError) as e:
            B.syr2k_lower(**args)
        assert e.value.code == code


@pytest.mark.parametrize("alpha,beta", [(1.0, 0.0), (-1.0, 1.0), (2.5, -0.5)])
def test_launch_forms_agree_bit_for_bit(alpha, beta):
    """One block per item and persistent blocks (whose write-out warps store C: a copy for beta = 0, a
    memory-side addition for beta = 1) run the same arithmetic: identical bits, both within tolerance."""
    for n, (N, M, ldc_pad) in enumerate([(40, 50, 0), (1000, 70, 0), (1300, 40, 3), (2500, 33, 0), (4100, 48, 2)]):
        A, Bm = I.normal_f64(N, M, seed=7000 + n), I.normal_f64(N, M, seed=7100 + n)
        Cin = I.random_c(N, 7200 + n, B.DTYPE_F64) if beta != 0.0 else None
        outs = []
        for mode in (B.F64_LAUNCH_PER_ITEM, B.F64_LAUNCH_PERSISTENT):
            try:
                B.syrk_set_f64_launch(mode)
                got, ref, bound = run(A, Bm, alpha, beta, Cin, ldc=N + ldc_pad, poison=(beta == 0.0))
            finally:
                B.syrk_set_f64_launch(B.F64_LAUNCH_AUTO)
            check(got, ref, bound, M, alpha, beta, Cin)
            outs.append(got)
        il = np.tril_indices(N)
        assert np.array_equal(outs[0][il], outs[1][il])
