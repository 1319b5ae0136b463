"""GPU parity of syr2k_lower_ex for the tcgen05 input types (bfloat16, binary16, TF32, FP8 E4M3; binary32
accumulation), through the C ABI, against the CPU reference of the rank-2k update on the decoded operands:

    |C_gpu - C_ref| <= 4 * 2^-24 * 2M * (|alpha| (|A||B|^T + |B||A|^T) + |beta| |C_in|)

(2M exact products per entry, summed in binary32); integer-valued inputs bit for bit; everything outside the
lower triangle bitwise untouched."""
import numpy as np
import pytest
import torch

from oracle import syr2k as R
from oracle import syrk as O
from paper_2202_10217_b200 import binding as B
from paper_2202_10217_b200 import inputs as I

from gpu_util import a_to_device, sentinel_array
from test_gpu_syrk import ALIGN_ELEMS, make_A

pytestmark = pytest.mark.gpu
TYPES = [B.DTYPE_BF16_F32, B.DTYPE_F16_F32, B.DTYPE_TF32_F32, B.DTYPE_E4M3_F32]
DT = pytest.mark.parametrize("dtype", TYPES, ids=["bf16", "f16", "tf32", "e4m3"])
GUARD = 3


def run(A, Bm, dtype, alpha, beta, Cin=None, lda=None, ldb=None, ldc=None, a_off=0, b_off=0, poison=False):
    N, M = A.shape
    ldc = max(N, 1) if ldc is None else ldc
    ka, pa = a_to_device(A, dtype, lda, a_off)
    kb, pb = a_to_device(Bm, dtype, ldb, b_off)
    host_c = sentinel_array((N + 2 * GUARD, ldc), np.float32)
    body = host_c[GUARD:GUARD + N, :N]
    il = np.tril_indices(N)
    if Cin is not None:
        body[il] = Cin[il]
    elif poison:
        body[il] = np.nan
    before = host_c.copy()
    dev_c = torch.from_numpy(host_c).cuda()
    B.syr2k_lower_ex(N, M, pa, max(M, 1) if lda is None else lda, pb, max(M, 1) if ldb is None else ldb,
                     dev_c.data_ptr() + 4 * GUARD * ldc, ldc, alpha, beta, dtype)
    torch.cuda.synchronize()
    assert B.syrk_last_status() == 0
    after = dev_c.cpu().numpy()
    mask = np.ones(after.shape, dtype=bool)
    mask[GUARD:GUARD + N, :N][il] = False
    assert np.array_equal(after.view(np.uint32)[mask], before.view(np.uint32)[mask]), "wrote outside the lower triangle"
    got = after[GUARD:GUARD + N, :N].astype(np.float64)
    ref, bound = R.syr2k_lower_typed(A, Bm, None if Cin is None else np.ascontiguousarray(Cin[:, :N]), alpha,
                                     beta if Cin is not None else 0.0, dtype)
    return got, ref, bound


def check(got, ref, bound, M, alpha, beta, Cin, exact=False):
    il = np.tril_indices(got.shape[0])
    g, r = got[il], ref[il]
    assert not np.isnan(g).any()
    if exact:
        assert np.array_equal(g, r), "max abs diff %g" % np.max(np.abs(g - r))
        return
    tol = R.tolerance(M, bound[il], None if Cin is None else np.abs(Cin[il].astype(np.float64)), alpha, beta, f32_accumulate=True)
    err = np.abs(g - r)
    assert np.all(err <= tol), "%d entries out of tolerance, worst ratio %g" % (int((err > tol).sum()), float(np.max(err / np.maximum(tol, 1e-300))))


SIZES = [(1, 16), (5, 48), (127, 128), (129, 144), (300, 400), (777, 272), (1100, 640), (2050, 144)]


@pytest.fixture(autouse=True)
def triangle_blocks():
    B.syrk_set_schedule(B.SCHEDULE_TBS)
    yield
    B.syrk_set_schedule(B.SCHEDULE_DEFAULT)


@DT
def test_real_and_integer_inputs(dtype):
    for n, (N, M) in enumerate(SIZES):
        A, Bm = make_A(N, M, dtype, seed=9300 + n), make_A(N, M, dtype, seed=9350 + n)
        got, ref, bound = run(A, Bm, dtype, 1.0, 0.0)
        check(got, ref, bound, M, 1.0, 0.0, None)
        Ai, Bi = make_A(N, M, dtype, seed=9400 + n, kind="int"), make_A(N, M, dtype, seed=9450 + n, kind="int")
        got, ref, bound = run(Ai, Bi, dtype, 1.0, 0.0, poison=True)
        check(got, ref, bound, M, 1.0, 0.0, None, exact=True)


@DT
@pytest.mark.parametrize("alpha,beta", [(-1.0, 1.0), (2.5, -0.5), (0.0, 2.0), (0.0, 0.0)])
def test_alpha_beta_pitches_and_offsets(dtype, alpha, beta):
    N, M = 900, 256
    step = ALIGN_ELEMS[dtype]
    A, Bm = make_A(N, M, dtype, seed=9500), make_A(N, M, dtype, seed=9501)
    Cin = I.random_c(N, 9502, dtype, ldc=N + 7)
    got, ref, bound = run(A, Bm, dtype, alpha, beta, Cin, lda=M + 4 * step, ldb=M + 2 * step, ldc=N + 7, a_off=3 * step, b_off=step)
    if alpha == 0.0:
        il = np.tril_indices(N)
        assert np.array_equal(got[il], (np.float32(beta) * Cin[:, :N][il]).astype(np.float64))
        return
    check(got, ref, bound, M, alpha, beta, Cin[:, :N])


@DT
def test_b_equal_a_is_twice_the_rank_k_update_and_exchange_changes_nothing(dtype):
    N, M = 1000, 320
    A, Bm = make_A(N, M, dtype, seed=9600, kind="int"), make_A(N, M, dtype, seed=9601, kind="int")
    got, _, _ = run(A, A, dtype, 1.0, 0.0)
    once, _ = O.syrk_lower(A, None, 1.0, 0.0, dtype)
    il = np.tril_indices(N)
    assert np.array_equal(got[il], 2.0 * once[il])
    ab, _, _ = run(A, Bm, dtype, 1.0, 0.0)
    ba, _, _ = run(Bm, A, dtype, 1.0, 0.0)
    assert np.array_equal(ab[il], ba[il])


@DT
@pytest.mark.parametrize("split", [2, 5])
def test_forced_k_split_and_square_schedule(dtype, split):
    N, M = 800, 2560
    A, Bm = make_A(N, M, dtype, seed=9700, kind="int"), make_A(N, M, dtype, seed=9701, kind="int")
    Cin = np.round(I.random_c(N, 9702, dtype) * 4).astype(np.float32)
    try:
        B.syrk_set_split_k(split)
        got, ref, bound = run(A, Bm, dtype, 1.0, -1.0, Cin)
    finally:
        B.syrk_set_split_k(0)
    check(got, ref, bound, M, 1.0, -1.0, Cin, exact=True)
    try:
        B.syrk_set_schedule(B.SCHEDULE_SQUARE)
        got, ref, bound = run(A, Bm, dtype, 1.0, -1.0, Cin)
    finally:
        B.syrk_set_schedule(B.SCHEDULE_TBS)
    check(got, ref, bound, M, 1.0, -1.0, Cin, exact=True)


@DT
def test_unaligned_operands_take_the_plain_kernel(dtype):
    N, M = 150, 77
    A, Bm = make_A(N, M, dtype, seed=9800), make_A(N, M, dtype, seed=9801)
    Cin = I.random_c(N, 9802, dtype)
    got, ref, bound = run(A, Bm, dtype, 1.5, 0.5, Cin, lda=M + 3, a_off=1)
    check(got, ref, bound, M, 1.5, 0.5, Cin)
    got, ref, bound = run(A, Bm, dtype, 1.5, 0.5, Cin, ldb=M + 1, b_off=3)
    check(got, ref, bound, M, 1.5, 0.5, Cin)


def test_large_size_sampled_and_argument_errors():
    N, M, dtype = 8192, 2048, B.DTYPE_BF16_F32
    A, Bm = make_A(N, M, dtype, seed=9900), make_A(N, M, dtype, seed=9901)
    ka, pa = a_to_device(A, dtype)
    kb, pb = a_to_device(Bm, dtype)
    dC = torch.full((N, N), float("nan"), dtype=torch.float32, device="cuda")
    B.syr2k_lower_ex(N, M, pa, M, pb, M, dC, N, 1.0, 0.0, dtype)
    torch.cuda.synchronize()
    assert B.syrk_last_status() == 0
    nan_mask = torch.isnan(dC)
    assert bool(torch.equal(nan_mask, torch.triu(torch.ones_like(nan_mask), diagonal=1)))
    rng = np.random.default_rng(9902)
    ii = rng.integers(0, N, size=4000)
    jj = (rng.random(4000) * (ii + 1)).astype(np.int64)
    got = dC[torch.from_numpy(ii).cuda(), torch.from_numpy(jj).cuda()].cpu().numpy().astype(np.float64)
    A64, B64 = O.widen(A, dtype), O.widen(Bm, dtype)
    ref = np.einsum("pk,pk->p", A64[ii], B64[jj]) + np.einsum("pk,pk->p", B64[ii], A64[jj])
    bound = np.einsum("pk,pk->p", np.abs(A64[ii]), np.abs(B64[jj])) + np.einsum("pk,pk->p", np.abs(B64[ii]), np.abs(A64[jj]))
    assert np.all(np.abs(got - ref) <= R.tolerance(M, bound, None, 1.0, 0.0, f32_accumulate=True))
    with pytest.raises(B.SyrkError):
        B.syr2k_lower_ex(8, 8, pa, 4, pb, 8, dC, N, 1.0, 0.0, dtype)            # lda < M
    with pytest.raises(B.SyrkError):
        B.syr2k_lower_ex(8, 8, pa, 8, None, 8, dC, N, 1.0, 0.0, dtype)          # null B
    with pytest.raises(B.SyrkError):
        B.syr2k_lower_ex(8, 8, pa, 8, pb, 8, dC, N, 1.0, 0.0, 9)                # unknown dtype
