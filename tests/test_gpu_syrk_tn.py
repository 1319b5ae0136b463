"""GPU parity of the Gram form C = alpha * A^T A + beta * C (A stored M x N row-major),
through syrk_lower_tn, against the same CPU reference as the N x M form: the reference is
Algorithm 1 applied to the N x M matrix A^T, so it receives the transposed array.
Tolerances as in test_gpu_syrk.py; integer-valued inputs must match bit for bit.
"""
import numpy as np
import pytest

from oracle import syrk as O
from paper_2202_10217_b200 import binding as B
from paper_2202_10217_b200 import inputs as I

from gpu_util import assert_within_tolerance, run_case
from test_gpu_syrk import make_A

pytestmark = pytest.mark.gpu
BOTH = [B.DTYPE_F64, B.DTYPE_BF16_F32, B.DTYPE_F16_F32, B.DTYPE_TF32_F32, B.DTYPE_E4M3_F32]
DT = pytest.mark.parametrize("dtype", BOTH, ids=["f64", "bf16", "f16", "tf32", "e4m3"])

# N even keeps the pitch of the M x N array a multiple of 16 bytes (tensor-core path in FP64);
# odd N takes the plain-load kernel.  Ragged tiles in N (not a multiple of 32) and ragged
# K-steps (M not a multiple of 16) are both covered.
SIZES = {B.DTYPE_F64: [(2, 1), (6, 3), (30, 17), (32, 16), (34, 50), (100, 64), (258, 130), (512, 256),
                       (1000, 70), (1300, 40), (2500, 33), (33, 20), (257, 19)],
         B.DTYPE_BF16_F32: [(8, 8), (40, 24), (128, 64), (136, 72), (304, 200), (777, 136), (512, 256),
                            (1104, 320), (2056, 72), (1304, 1000)]}
SIZES[B.DTYPE_F16_F32] = SIZES[B.DTYPE_BF16_F32]
SIZES[B.DTYPE_TF32_F32] = [(4, 4), (40, 12), (128, 32), (132, 36), (304, 100), (777, 68), (512, 256), (1100, 160),
                           (2052, 44), (1304, 500)]
SIZES[B.DTYPE_E4M3_F32] = [(16, 16), (48, 48), (128, 128), (144, 272), (304, 400), (777, 144), (512, 512),
                           (1104, 640), (2064, 144), (1312, 1008)]


@DT
def test_real_inputs_within_tolerance(dtype):
    for n, (N, M) in enumerate(SIZES[dtype]):
        A = make_A(N, M, dtype, seed=400 + n)
        got, ref, bound = run_case(A, dtype, 1.0, 0.0, tn=True)
        assert_within_tolerance(got, ref, bound, M, 1.0, 0.0, None, dtype)


@DT
def test_integer_inputs_are_bit_exact(dtype):
    for n, (N, M) in enumerate(SIZES[dtype]):
        A = make_A(N, M, dtype, seed=500 + n, kind="int")
        got, ref, bound = run_case(A, dtype, 1.0, 0.0, tn=True)
        assert_within_tolerance(got, ref, bound, M, 1.0, 0.0, None, dtype, exact=True)


@DT
@pytest.mark.parametrize("alpha,beta", [(-1.0, 1.0), (0.0, 1.0), (0.0, 0.0), (2.5, -0.5), (1.0, 2.0)])
def test_alpha_beta(dtype, alpha, beta):
    N, M = (1100, 48) if dtype == B.DTYPE_F64 else (520, 72)
    A = make_A(N, M, dtype, seed=21, kind="int")
    Cin = I.random_c(N, 22, dtype)
    got, ref, bound = run_case(A, dtype, alpha, beta, Cin, tn=True)
    assert_within_tolerance(got, ref, bound, M, alpha, beta, Cin, dtype)


@DT
def test_pitches_offsets_and_nan_poison(dtype):
    N, M = (300, 45) if dtype == B.DTYPE_F64 else (264, 90)
    A = make_A(N, M, dtype, seed=23)
    Cin = I.random_c(N, 24, dtype)
    got, ref, bound = run_case(A, dtype, -1.0, 1.0, Cin, lda=N + 24, ldc=N + 10, a_offset=8, c_offset=6, tn=True)
    assert_within_tolerance(got, ref, bound, M, -1.0, 1.0, Cin, dtype)
    got, ref, bound = run_case(A, dtype, 1.0, 0.0, poison=True, tn=True)      # beta = 0: C is not read
    assert_within_tolerance(got, ref, bound, M, 1.0, 0.0, None, dtype)


def test_unaligned_operand_takes_the_plain_kernel():
    N, M = 200, 37
    A = make_A(N, M, B.DTYPE_F64, seed=25, kind="int")
    got, ref, bound = run_case(A, B.DTYPE_F64, 1.0, 0.0, lda=N + 1, a_offset=1, tn=True)
    assert_within_tolerance(got, ref, bound, M, 1.0, 0.0, None, B.DTYPE_F64, exact=True)


def test_both_launch_forms_agree_bit_for_bit_in_this_storage_order():
    """FP64: one block per item and persistent blocks run every tile with the same arithmetic in
    the same order, so their results are identical; each is within tolerance of the reference."""
    for n, (N, M) in enumerate([(1000, 70), (2500, 33), (5000, 48)]):
        A = make_A(N, M, B.DTYPE_F64, seed=600 + n)
        Cin = I.random_c(N, 9, B.DTYPE_F64)
        outs = []
        for mode in (B.F64_LAUNCH_PER_ITEM, B.F64_LAUNCH_PERSISTENT):
            try:
                B.syrk_set_f64_launch(mode)
                got, ref, bound = run_case(A, B.DTYPE_F64, -1.0, 1.0, Cin, tn=True)
            finally:
                B.syrk_set_f64_launch(B.F64_LAUNCH_AUTO)
            assert_within_tolerance(got, ref, bound, M, -1.0, 1.0, Cin, B.DTYPE_F64)
            outs.append(got)
        il = np.tril_indices(N)
        assert np.array_equal(outs[0][il], outs[1][il])


def test_leading_dimension_smaller_than_N_is_refused():
    with pytest.raises(Exception):
        B.syrk_lower_tn(64, 16, 8, 32, 8, 64, 1.0, 0.0, B.DTYPE_F64, stream=0)


@pytest.mark.parametrize("dtype", [B.DTYPE_BF16_F32, B.DTYPE_F16_F32, B.DTYPE_TF32_F32, B.DTYPE_E4M3_F32],
                         ids=["bf16", "f16", "tf32", "e4m3"])
@pytest.mark.parametrize("split", [0, 2, 5])
def test_bf16_k_split_in_this_storage_order(split, dtype):
    N, M = 704, 1280
    A = make_A(N, M, dtype, seed=40 + split, kind="int")
    Cin = I.random_c(N, 41, dtype)
    try:
        B.syrk_set_split_k(split)
        got, ref, bound = run_case(A, dtype, 2.0, -1.0, Cin, tn=True)
    finally:
        B.syrk_set_split_k(0)
    assert_within_tolerance(got, ref, bound, M, 2.0, -1.0, Cin, dtype)


def test_tf32_low_order_bits_are_ignored_in_this_storage_order():
    """The MN-major TF32 path reads the same 19 high-order bits as the N x M path."""
    N, M = 264, 96
    base = I.small_int_f32(N, M, seed=63, lo=-3, hi=3)
    noise = np.random.default_rng(64).integers(0, 1 << 13, size=base.shape, dtype=np.uint32)
    dirty = (base.view(np.uint32) | np.where(base != 0, noise, 0).astype(np.uint32)).view(np.float32)
    got_dirty, ref, bound = run_case(dirty, B.DTYPE_TF32_F32, 1.0, 0.0, tn=True)
    got_clean, _, _ = run_case(base, B.DTYPE_TF32_F32, 1.0, 0.0, tn=True)
    il = np.tril_indices(N)
    assert np.array_equal(got_dirty[il], got_clean[il]) and np.array_equal(got_dirty[il], ref[il])
