"""GPU parity of the strided batch entry point syrk_lower_batched: every matrix of the batch against
the CPU reference (Algorithm 1 applied to that matrix), entry by entry, under the tolerance of
test_gpu_syrk.py; integer-valued inputs bit for bit.  Everything between and around the lower
triangles (upper triangles, pitch padding, the gaps between matrices, guard elements) must stay
bitwise untouched.
"""
import numpy as np
import pytest
import torch

from oracle import syrk as O
from paper_2202_10217_b200 import binding as B
from paper_2202_10217_b200 import inputs as I

from gpu_util import a_to_device, assert_within_tolerance, sentinel_array
from test_gpu_syrk import ALIGN_ELEMS, BOTH, make_A

pytestmark = pytest.mark.gpu
DT = pytest.mark.parametrize("dtype", BOTH, ids=["f64", "bf16", "tf32", "e4m3", "f16"])
GUARD = 7            # sentinel elements before the first and after the last matrix of C


def run_batched(As, dtype, alpha, beta, Cins=None, lda=None, ldc=None, stride_a=None, stride_c=None,
                poison=False):
    """One syrk_lower_batched call on the matrices `As` (all N x M); returns the list of results.
    Checks status and that nothing outside the lower triangles was written."""
    batch = len(As)
    N, M = As[0].shape
    lda = max(M, 1) if lda is None else lda
    ldc = max(N, 1) if ldc is None else ldc
    stride_a = N * lda if stride_a is None else stride_a
    stride_c = N * ldc if stride_c is None else stride_c
    cdt = I.c_storage_dtype(dtype)
    # A: one buffer holding every matrix at its stride
    host_a = np.zeros(batch * stride_a + lda, dtype=As[0].dtype)
    for b, A in enumerate(As):
        view = host_a[b * stride_a: b * stride_a + N * lda].reshape(N, lda)
        view[:, :M] = A
    keep, a_ptr = a_to_device(host_a.reshape(1, -1), dtype)
    # C: sentinels everywhere, prior values (or NaN) in the lower triangles
    host_c = sentinel_array((GUARD + batch * stride_c + ldc + GUARD,), cdt)
    il = np.tril_indices(N)
    for b in range(batch):
        body = host_c[GUARD + b * stride_c: GUARD + b * stride_c + N * ldc].reshape(N, ldc)[:, :N]
        if Cins is not None:
            body[il] = Cins[b][il]
        elif poison:
            body[il] = np.nan
    before = host_c.copy()
    dev_c = torch.from_numpy(host_c).cuda()
    c_ptr = dev_c.data_ptr() + GUARD * dev_c.element_size()
    B.syrk_lower_batched(batch, N, M, a_ptr, lda, stride_a, c_ptr, ldc, stride_c, alpha, beta, dtype)
    torch.cuda.synchronize()
    assert B.syrk_last_status() == 0
    after = dev_c.cpu().numpy()
    u = np.uint64 if cdt == np.float64 else np.uint32
    mask = np.ones(after.shape, dtype=bool)
    got = []
    for b in range(batch):
        lo = GUARD + b * stride_c
        m = mask[lo: lo + N * ldc].reshape(N, ldc)[:, :N]
        m[il] = False
        got.append(after[lo: lo + N * ldc].reshape(N, ldc)[:, :N].astype(np.float64))
    assert np.array_equal(after.view(u)[mask], before.view(u)[mask]), "wrote outside the lower triangles"
    return got


def check(As, got, dtype, alpha, beta, Cins=None, exact=False):
    M = As[0].shape[1]
    for b, A in enumerate(As):
        Cin = None if Cins is None else Cins[b]
        ref, bound = O.syrk_lower(np.ascontiguousarray(A), Cin, alpha, beta if Cin is not None else 0.0, dtype)
        try:
            assert_within_tolerance(got[b], ref, bound, M, alpha, beta, Cin, dtype, exact=exact)
        except AssertionError as e:
            raise AssertionError("matrix %d of %d: %s" % (b, len(As), e))


def shapes(dtype):
    """(batch, N, M): below one tile, ragged tiles and K-steps, several tiles, triangle-block sizes."""
    a = ALIGN_ELEMS[dtype]
    if dtype == B.DTYPE_F64:
        return [(3, 5, 4), (4, 33, 18), (7, 100, 64), (5, 257, 130), (160, 96, 32), (3, 1056, 48), (2, 1300, 40)]
    return [(3, 5, a), (4, 129, 9 * a), (6, 300, 25 * a), (5, 512, 256), (150, 136, 4 * a), (3, 1100, 20 * a),
            (2, 2050, 9 * a)]


@DT
def test_real_inputs_within_tolerance(dtype):
    for n, (batch, N, M) in enumerate(shapes(dtype)):
        As = [make_A(N, M, dtype, seed=2000 + 10 * n + b) for b in range(batch)]
        got = run_batched(As, dtype, 1.0, 0.0)
        check(As, got, dtype, 1.0, 0.0)


@DT
def test_integer_inputs_are_bit_exact(dtype):
    for n, (batch, N, M) in enumerate(shapes(dtype)[:6]):
        As = [make_A(N, M, dtype, seed=2500 + 10 * n + b, kind="int") for b in range(batch)]
        got = run_batched(As, dtype, 1.0, 0.0)
        check(As, got, dtype, 1.0, 0.0, exact=True)


@DT
@pytest.mark.parametrize("alpha,beta", [(-1.0, 1.0), (2.5, -0.5), (0.0, 0.5), (0.0, 0.0)])
def test_alpha_beta_pitches_and_gaps(dtype, alpha, beta):
    """General scalars, row pitches larger than the rows and gaps between the matrices (aligned)."""
    a = ALIGN_ELEMS[dtype]
    batch, N, M = (5, 200, 48) if dtype == B.DTYPE_F64 else (5, 264, 6 * a)
    lda, ldc = M + 2 * a, N + 12
    stride_a, stride_c = N * lda + 3 * a, N * ldc + 8
    As = [make_A(N, M, dtype, seed=2700 + b, kind="int") for b in range(batch)]
    Cins = [I.random_c(N, 2800 + b, dtype) for b in range(batch)]
    got = run_batched(As, dtype, alpha, beta, Cins, lda=lda, ldc=ldc, stride_a=stride_a, stride_c=stride_c)
    check(As, got, dtype, alpha, beta, Cins)


@DT
def test_beta_zero_ignores_nan_in_C(dtype):
    a = ALIGN_ELEMS[dtype]
    batch, N, M = 4, 140, 4 * a
    As = [make_A(N, M, dtype, seed=2900 + b) for b in range(batch)]
    got = run_batched(As, dtype, 1.0, 0.0, poison=True)
    check(As, got, dtype, 1.0, 0.0)


@DT
def test_unaligned_strides_take_the_one_by_one_path(dtype):
    """A matrix stride (or pitch, or an odd C stride) that breaks the 16-byte rules: same results."""
    a = ALIGN_ELEMS[dtype]
    batch, N, M = 3, 150, 5 * a
    As = [make_A(N, M, dtype, seed=3000 + b) for b in range(batch)]
    Cins = [I.random_c(N, 3100 + b, dtype) for b in range(batch)]
    got = run_batched(As, dtype, 1.5, 0.5, Cins, lda=M, stride_a=N * M + 1, ldc=N + 1, stride_c=N * (N + 1) + 3)
    check(As, got, dtype, 1.5, 0.5, Cins)
    # aligned A, odd C pitch and stride: the single launch with scalar stores
    got = run_batched(As, dtype, 1.5, 0.5, Cins, ldc=N + 1, stride_c=N * (N + 1) + 3)
    check(As, got, dtype, 1.5, 0.5, Cins)


def test_batch_of_one_and_of_zero_and_argument_errors():
    A = make_A(70, 16, B.DTYPE_F64, seed=3200)
    got = run_batched([A], B.DTYPE_F64, 1.0, 0.0)
    check([A], got, B.DTYPE_F64, 1.0, 0.0)
    dA = torch.zeros(4 * 70 * 16, dtype=torch.float64, device="cuda")
    dC = torch.full((4 * 70 * 70,), 3.0, dtype=torch.float64, device="cuda")
    B.syrk_lower_batched(0, 70, 16, dA, 16, 70 * 16, dC, 70, 70 * 70, 1.0, 0.0, B.DTYPE_F64)   # nothing to do
    torch.cuda.synchronize()
    assert bool((dC == 3.0).all())
    for kwargs, code in [(dict(batch=-1), -2), (dict(stride_a=70 * 16 - 1), -3), (dict(stride_c=70 * 70 - 1), -3),
                         (dict(lda=15), -3), (dict(dtype=99), -4)]:
        args = dict(batch=4, N=70, M=16, A=dA, lda=16, stride_a=70 * 16, C=dC, ldc=70, stride_c=70 * 70,
                    alpha=1.0, beta=0.0, dtype=B.DTYPE_F64)
        args.update(kwargs)
        with pytest.raises(B.SyrkError) as e:
            B.syrk_lower_batched(**args)
        assert e.value.code == code
    torch.cuda.synchronize()
    assert bool((dC == 3.0).all())


@pytest.mark.parametrize("alpha,beta", [(1.0, 0.0), (-1.0, 1.0), (2.5, -0.5)])
def test_f64_launch_forms_agree_bit_for_bit(alpha, beta):
    """FP64 batches on persistent blocks (tickets over the (matrix, item) pairs, C written by the write-out warps)
    against one block per (matrix, item): identical bits, both within tolerance; gaps between the matrices, an odd
    stride of C (8-byte accesses), and short inner dimensions (items of one to three K-steps)."""
    for n, (batch, N, M, c_gap) in enumerate([(40, 96, 32, 0), (300, 70, 20, 0), (9, 520, 100, 8), (6, 1056, 48, 3)]):
        As = [make_A(N, M, B.DTYPE_F64, seed=2900 + 10 * n + b) for b in range(batch)]
        Cins = [I.random_c(N, 2950 + 10 * n + b, B.DTYPE_F64) for b in range(batch)] if beta != 0.0 else None
        outs = []
        for mode in (B.F64_LAUNCH_PER_ITEM, B.F64_LAUNCH_PERSISTENT):
            try:
                B.syrk_set_f64_launch(mode)
                got = run_batched(As, B.DTYPE_F64, alpha, beta, Cins, stride_c=N * N + c_gap, poison=(beta == 0.0))
            finally:
                B.syrk_set_f64_launch(B.F64_LAUNCH_AUTO)
            check(As, got, B.DTYPE_F64, alpha, beta, Cins)
            outs.append(got)
        il = np.tril_indices(N)
        for b in range(batch):
            assert np.array_equal(outs[0][b][il], outs[1][b][il]), (n, b)
