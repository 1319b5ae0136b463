"""Seeded random sweep of the C-ABI surface on the GPU: every input type, both storage orders
of the operand, both stored triangles, aligned and unaligned bases and pitches, general alpha / beta, forced K-splits and
both FP64 launch forms - each case compared entry by entry with the CPU reference under the
tolerance of test_gpu_syrk.py (and bit for bit when the inputs are small integers)."""
import numpy as np
import pytest

from paper_2202_10217_b200 import binding as B
from paper_2202_10217_b200 import inputs as I

from gpu_util import assert_within_tolerance, run_case
from test_gpu_syrk import ALIGN_ELEMS, make_A

pytestmark = pytest.mark.gpu

DTYPES = [B.DTYPE_F64, B.DTYPE_BF16_F32, B.DTYPE_TF32_F32, B.DTYPE_E4M3_F32, B.DTYPE_F16_F32]
SCALARS = [(1.0, 0.0), (-1.0, 1.0), (0.5, -2.0), (2.0, 0.0), (1.0, 1.0), (0.0, 0.5)]


@pytest.mark.parametrize("chunk", range(8))
def test_random_cases(chunk):
    rng = np.random.default_rng(9000 + chunk)
    for case in range(12):
        dtype = DTYPES[int(rng.integers(0, len(DTYPES)))]
        tn = bool(rng.integers(0, 2))
        upper = bool(rng.integers(0, 3) == 0)
        kind = "int" if rng.integers(0, 3) == 0 else "normal"
        N = int(rng.choice([int(rng.integers(1, 130)), int(rng.integers(130, 700)), int(rng.integers(700, 1700))]))
        M = int(rng.choice([int(rng.integers(1, 40)), int(rng.integers(40, 300)), int(rng.integers(300, 900))]))
        alpha, beta = SCALARS[int(rng.integers(0, len(SCALARS)))]
        align = ALIGN_ELEMS[dtype]
        inner = N if tn else M                                  # contiguous extent of the stored operand
        if rng.integers(0, 4) == 0:                             # unaligned base or pitch: plain-load kernel
            lda, a_offset = inner + int(rng.integers(0, 5)), int(rng.integers(0, 3))
        else:                                                   # 16-byte aligned: TMA kernels
            lda = (inner + align - 1) // align * align + align * int(rng.integers(0, 3))
            a_offset = align * int(rng.integers(0, 3))
        ldc, c_offset = N + int(rng.integers(0, 9)), int(rng.integers(0, 4))
        A = make_A(N, M, dtype, seed=int(rng.integers(0, 1 << 30)), kind=kind)
        Cin = I.random_c(N, int(rng.integers(0, 1 << 30)), dtype) if beta != 0.0 else None
        if Cin is not None and kind == "int":
            Cin = np.round(Cin * 4).astype(Cin.dtype)           # keeps every partial result exact
        split = int(rng.choice([0, 0, 2, 3]))
        mode = int(rng.integers(0, 3)) if dtype == B.DTYPE_F64 else 0
        try:
            B.syrk_set_split_k(split)
            B.syrk_set_f64_launch(mode)
            got, ref, bound = run_case(A, dtype, alpha, beta, Cin, lda=lda, ldc=ldc, a_offset=a_offset,
                                       c_offset=c_offset, tn=tn, upper=upper)
        finally:
            B.syrk_set_split_k(0)
            B.syrk_set_f64_launch(B.F64_LAUNCH_AUTO)
        where = "case %d.%d dtype=%d tn=%s upper=%s N=%d M=%d lda=%d off=%d a=%g b=%g split=%d mode=%d" % (
            chunk, case, dtype, tn, upper, N, M, lda, a_offset, alpha, beta, split, mode)
        try:
            exact = kind == "int" and float(alpha).is_integer() and float(beta).is_integer()
            assert_within_tolerance(got, ref, bound, M, alpha, beta, Cin, dtype, exact=exact)
        except AssertionError as e:
            raise AssertionError(where + ": " + str(e))
