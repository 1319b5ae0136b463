"""GPU parity of the CTA-pair square-block schedule (SYRK_SCHEDULE_PAIR_SQUARE: 256 x 256 blocks on pairs
of thread blocks) against the CPU reference, for the four
tcgen05 input types: sizes with an even and an odd number of tile rows, ragged last tiles and K-steps,
integer inputs bit for bit, general alpha / beta with pitches, NaN-poisoned C with beta = 0; the calls
the schedule does not cover (small problems, the other storage order, the other types) must fall back
and still match."""
import numpy as np
import pytest

from paper_2202_10217_b200 import binding as B
from paper_2202_10217_b200 import inputs as I

from gpu_util import assert_within_tolerance, run_case
from test_gpu_syrk import make_A

pytestmark = pytest.mark.gpu
DT = pytest.mark.parametrize("dtype", [B.DTYPE_BF16_F32, B.DTYPE_F16_F32, B.DTYPE_TF32_F32, B.DTYPE_E4M3_F32],
                         ids=["bf16", "f16", "tf32", "e4m3"])


@pytest.fixture(autouse=True)
def pair_schedule():
    B.syrk_set_schedule(B.SCHEDULE_PAIR_SQUARE)
    yield
    B.syrk_set_schedule(B.SCHEDULE_DEFAULT)


SIZES = [(3200, 144), (3328, 64), (4200, 320)]      # M: multiples of 16 bytes for every type


@DT
def test_real_inputs_within_tolerance(dtype):
    for n, (N, M) in enumerate(SIZES):
        A = make_A(N, M, dtype, seed=7000 + n)
        got, ref, bound = run_case(A, dtype, 1.0, 0.0)
        assert_within_tolerance(got, ref, bound, M, 1.0, 0.0, None, dtype)


@DT
def test_integer_inputs_are_bit_exact(dtype):
    for n, (N, M) in enumerate(SIZES):
        A = make_A(N, M, dtype, seed=7100 + n, kind="int")
        got, ref, bound = run_case(A, dtype, 1.0, 0.0)
        assert_within_tolerance(got, ref, bound, M, 1.0, 0.0, None, dtype, exact=True)


@DT
@pytest.mark.parametrize("alpha,beta", [(2.5, -0.5), (1.0, 0.0)])
def test_alpha_beta_pitches_and_poison(dtype, alpha, beta):
    N, M = 3300, 112
    A = make_A(N, M, dtype, seed=7200, kind="int")
    Cin = I.random_c(N, 7201, dtype)
    got, ref, bound = run_case(A, dtype, alpha, beta, Cin if beta != 0.0 else None, lda=M + 16, ldc=N + 12,
                               a_offset=16, c_offset=4, poison=(beta == 0.0))
    assert_within_tolerance(got, ref, bound, M, alpha, beta, Cin if beta != 0.0 else None, dtype)
    got, ref, bound = run_case(A, dtype, alpha, beta, Cin if beta != 0.0 else None, ldc=N + 3)   # odd pitch: scalar stores
    assert_within_tolerance(got, ref, bound, M, alpha, beta, Cin if beta != 0.0 else None, dtype)


@DT
def test_k_split_automatic_and_forced(dtype):
    """Few blocks and a long inner dimension: (block, K-slice) units with partial tiles summed in slice order.
    Automatic choice at 2048 x 8192 and 1100 x 8208 (odd number of tile rows, ragged last K-step); forced
    2 and 7 slices at a size that needs none; integer inputs bit for bit."""
    for n, (N, M) in enumerate([(2048, 8192), (1100, 8208)]):
        A = make_A(N, M, dtype, seed=7400 + n, kind="int")
        Cin = np.round(I.random_c(N, 7401, dtype) * 4).astype(np.float32)
        got, ref, bound = run_case(A, dtype, 1.0, -1.0, Cin)
        assert_within_tolerance(got, ref, bound, M, 1.0, -1.0, Cin, dtype, exact=True)
        A = make_A(N, M, dtype, seed=7410 + n)
        got, ref, bound = run_case(A, dtype, 0.5, 0.0, poison=True)
        assert_within_tolerance(got, ref, bound, M, 0.5, 0.0, None, dtype)
    for split in (2, 7):
        A = make_A(3200, 1296, dtype, seed=7420 + split)
        Cin = I.random_c(3200, 7421, dtype)
        try:
            B.syrk_set_split_k(split)
            got, ref, bound = run_case(A, dtype, -1.0, 1.0, Cin, ldc=3203)
        finally:
            B.syrk_set_split_k(0)
        assert_within_tolerance(got, ref, bound, 1296, -1.0, 1.0, Cin, dtype)


def test_calls_outside_the_schedule_fall_back():
    for dtype, N, M, tn, upper in [(B.DTYPE_BF16_F32, 700, 72, False, False), (B.DTYPE_BF16_F32, 3200, 72, True, False),
                                   (B.DTYPE_F16_F32, 3200, 72, False, True), (B.DTYPE_F64, 1100, 48, False, False),
                                   (B.DTYPE_E4M3_F32, 3200, 136, False, False)]:
        A = make_A(N, M, dtype, seed=7300)
        got, ref, bound = run_case(A, dtype, 1.0, 0.0, tn=tn, upper=upper)
        assert_within_tolerance(got, ref, bound, M, 1.0, 0.0, None, dtype)


def test_automatic_schedule():
    """SYRK_SCHEDULE_AUTO: triangle blocks, except for lists shorter than a few rounds of SMs (the sizes an
    entry-by-entry reference can check all fall there; the long-list branch is the default schedule, covered by
    every other test file).  Integer inputs bit for bit."""
    try:
        B.syrk_set_schedule(B.SCHEDULE_AUTO)
        for dtype, N, M in [(B.DTYPE_BF16_F32, 1536, 8192), (B.DTYPE_E4M3_F32, 2048, 8192),      # short lists, K-split: pairs
                            (B.DTYPE_BF16_F32, 3200, 144), (B.DTYPE_F64, 1100, 48)]:           # pairs without K-split / FP64: triangle blocks
            A = make_A(N, M, dtype, seed=7500, kind="int")
            Cin = np.round(I.random_c(N, 7501, dtype) * 4).astype(I.c_storage_dtype(dtype))
            got, ref, bound = run_case(A, dtype, 1.0, -1.0, Cin)
            assert_within_tolerance(got, ref, bound, M, 1.0, -1.0, Cin, dtype, exact=True)
    finally:
        B.syrk_set_schedule(B.SCHEDULE_PAIR_SQUARE)      # what the fixture of this file expects to undo
