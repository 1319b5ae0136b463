"""GPU parity of syrk_ex with the UPPER triangle stored, in both storage orders of the operand, against
the CPU reference: Algorithm 1 gives a symmetric C, so entry (j, i) of the upper form must equal the
reference's entry (i, j) under the tolerance of test_gpu_syrk.py (bit for bit on integer inputs), and
nothing outside the upper triangle may be touched.  The lower form of syrk_ex must be syrk_lower bit for bit.
"""
import numpy as np
import pytest
import torch

from paper_2202_10217_b200 import binding as B
from paper_2202_10217_b200 import inputs as I

from gpu_util import assert_within_tolerance, run_case
from test_gpu_syrk import ALIGN_ELEMS, BOTH, make_A, sizes

pytestmark = pytest.mark.gpu
DT = pytest.mark.parametrize("dtype", BOTH, ids=["f64", "bf16", "tf32", "e4m3", "f16"])
TN = pytest.mark.parametrize("tn", [False, True], ids=["nxm", "mxn"])


def tn_sizes(dtype):
    """N a multiple of 16 bytes of elements so that the M x N operand takes the tensor-core path."""
    a = ALIGN_ELEMS[dtype]
    return [((N + a - 1) // a * a, M) for N, M in sizes(dtype)]


@DT
@TN
def test_real_inputs_within_tolerance(dtype, tn):
    for n, (N, M) in enumerate(tn_sizes(dtype) if tn else sizes(dtype)):
        A = make_A(N, M, dtype, seed=4000 + n)
        got, ref, bound = run_case(A, dtype, 1.0, 0.0, tn=tn, upper=True)
        assert_within_tolerance(got, ref, bound, M, 1.0, 0.0, None, dtype)


@DT
@TN
def test_integer_inputs_are_bit_exact(dtype, tn):
    for n, (N, M) in enumerate(tn_sizes(dtype) if tn else sizes(dtype)):
        A = make_A(N, M, dtype, seed=4100 + n, kind="int")
        got, ref, bound = run_case(A, dtype, 1.0, 0.0, tn=tn, upper=True)
        assert_within_tolerance(got, ref, bound, M, 1.0, 0.0, None, dtype, exact=True)


@DT
@pytest.mark.parametrize("alpha,beta", [(-1.0, 1.0), (0.0, 1.0), (0.0, 0.0), (2.5, -0.5)])
def test_alpha_beta_pitches_offsets(dtype, alpha, beta):
    a = ALIGN_ELEMS[dtype]
    N, M = (1100, 48) if dtype == B.DTYPE_F64 else (520, 9 * a)
    A = make_A(N, M, dtype, seed=4200, kind="int")
    Cin = I.random_c(N, 4201, dtype)
    got, ref, bound = run_case(A, dtype, alpha, beta, Cin, lda=M + 2 * a, ldc=N + 10, a_offset=a, c_offset=6, upper=True)
    assert_within_tolerance(got, ref, bound, M, alpha, beta, Cin, dtype)
    got, ref, bound = run_case(A, dtype, alpha, beta, Cin, ldc=N + 3, upper=True)        # odd pitch: scalar stores
    assert_within_tolerance(got, ref, bound, M, alpha, beta, Cin, dtype)


@DT
def test_beta_zero_ignores_nan_and_unaligned_operand(dtype):
    N, M = 300, 5 * ALIGN_ELEMS[dtype]
    A = make_A(N, M, dtype, seed=4300)
    got, ref, bound = run_case(A, dtype, 1.0, 0.0, poison=True, upper=True)
    assert_within_tolerance(got, ref, bound, M, 1.0, 0.0, None, dtype)
    got, ref, bound = run_case(A, dtype, 1.0, 0.0, lda=M + 3, a_offset=1, upper=True)     # plain-load kernel
    assert_within_tolerance(got, ref, bound, M, 1.0, 0.0, None, dtype)


@DT
@TN
@pytest.mark.parametrize("split", [2, 5])
def test_k_split(dtype, tn, split):
    a = ALIGN_ELEMS[dtype]
    N, M = (258, 1030) if dtype == B.DTYPE_F64 else (704, 160 * a)
    A = make_A(N, M, dtype, seed=4400 + split, kind="int")
    Cin = I.random_c(N, 4401, dtype)
    try:
        B.syrk_set_split_k(split)
        got, ref, bound = run_case(A, dtype, 2.0, -1.0, Cin, tn=tn, upper=True)
    finally:
        B.syrk_set_split_k(0)
    assert_within_tolerance(got, ref, bound, M, 2.0, -1.0, Cin, dtype)


def test_large_triangle_block_sizes_and_square_schedule():
    """Sizes with many triangle blocks (FP64: the 16th-warp path in its mirrored form), and the
    square-block comparison schedule."""
    for dtype, N, M in [(B.DTYPE_F64, 2100, 70), (B.DTYPE_BF16_F32, 4200, 136)]:
        A = make_A(N, M, dtype, seed=4500)
        Cin = I.random_c(N, 4501, dtype)
        got, ref, bound = run_case(A, dtype, -1.0, 1.0, Cin, upper=True)
        assert_within_tolerance(got, ref, bound, M, -1.0, 1.0, Cin, dtype)
        try:
            B.syrk_set_schedule(B.SCHEDULE_SQUARE)
            got2, _, _ = run_case(A, dtype, -1.0, 1.0, Cin, upper=True)
        finally:
            B.syrk_set_schedule(B.SCHEDULE_DEFAULT)
        assert_within_tolerance(got2, ref, bound, M, -1.0, 1.0, Cin, dtype)


def test_lower_form_of_syrk_ex_is_syrk_lower_and_bad_flags_are_refused():
    N, M = 600, 96
    A = torch.from_numpy(make_A(N, M, B.DTYPE_F64, seed=4600)).cuda()
    C1 = torch.zeros((N, N), dtype=torch.float64, device="cuda")
    C2 = torch.zeros((N, N), dtype=torch.float64, device="cuda")
    B.syrk_lower(N, M, A, M, C1, N, 1.0, 0.0, B.DTYPE_F64)
    B.syrk_ex(B.UPLO_LOWER, B.OP_N, N, M, A, M, C2, N, 1.0, 0.0, B.DTYPE_F64)
    torch.cuda.synchronize()
    assert torch.equal(C1, C2)
    for uplo, trans in [(2, 0), (0, 2), (-1, 0)]:
        with pytest.raises(B.SyrkError) as e:
            B.syrk_ex(uplo, trans, N, M, A, M, C2, N, 1.0, 0.0, B.DTYPE_F64)
        assert e.value.code == -2


@TN
@pytest.mark.parametrize("alpha,beta", [(1.0, 0.0), (-1.0, 1.0), (2.5, -0.5)])
def test_f64_launch_forms_agree_bit_for_bit_on_the_upper_triangle(tn, alpha, beta):
    """The persistent FP64 form (write-out by separate warps) with the upper triangle stored: same bits as the
    one-block-per-item form, within tolerance of the reference, ragged last tile row and column, odd pitch of C."""
    for n, (N, M, pad) in enumerate([(1304, 40, 0), (2500, 33, 3), (5008, 48, 0)]):
        if tn and N % 2:
            continue
        A = make_A(N, M, B.DTYPE_F64, seed=4500 + n)
        Cin = I.random_c(N, 4501, B.DTYPE_F64) if beta != 0.0 else None
        outs = []
        for mode in (B.F64_LAUNCH_PER_ITEM, B.F64_LAUNCH_PERSISTENT):
            try:
                B.syrk_set_f64_launch(mode)
                got, ref, bound = run_case(A, B.DTYPE_F64, alpha, beta, Cin, ldc=N + pad, tn=tn, upper=True,
                                           poison=(beta == 0.0))
            finally:
                B.syrk_set_f64_launch(B.F64_LAUNCH_AUTO)
            assert_within_tolerance(got, ref, bound, M, alpha, beta, Cin, B.DTYPE_F64)
            outs.append(got)
        il = np.tril_indices(N)
        assert np.array_equal(outs[0][il], outs[1][il])
