"""The allocation-free K-split entry point against the regular one.

syrk_lower_bf16_static is for callers that cannot let the library call cudaMalloc; it
keeps its work list and partial tiles in fixed device arrays.  Its result must agree
with syrk_lower (same K-split) within the BF16 parity tolerance, on two calls in a
row with different problems (the second call reuses the arrays the first one wrote).
Collected last, so that a failure here cannot hide another test's result.
"""
import numpy as np
import pytest
import torch

from oracle import syrk as O
from paper_2202_10217_b200 import binding as B
from paper_2202_10217_b200 import inputs as I

pytestmark = pytest.mark.gpu


def regular(A, Cin, alpha, beta, slices):
    N, M = A.shape
    dA = torch.from_numpy(A.view(np.int16)).cuda().view(torch.bfloat16)
    dC = torch.from_numpy(Cin.copy()).cuda()
    try:
        B.syrk_set_split_k(slices)
        B.syrk_lower(N, M, dA, M, dC, N, alpha, beta, B.DTYPE_BF16_F32)
        torch.cuda.synchronize()
    finally:
        B.syrk_set_split_k(0)
    assert B.syrk_last_status() == 0
    return dC.cpu().numpy()


def static(A, Cin, alpha, beta, slices):
    N, M = A.shape
    dA = torch.from_numpy(A.view(np.int16)).cuda().view(torch.bfloat16)
    dC = torch.from_numpy(Cin.copy()).cuda()
    B.syrk_lower_bf16_static(N, M, dA, M, dC, N, alpha, beta, slices)
    torch.cuda.synchronize()
    return dC.cpu().numpy()


def test_static_entry_point_matches_regular_one_twice_in_a_row():
    cases = [(1500, 2048, 4, 1.0, 0.0, 21), (900, 1280, 6, -1.0, 1.0, 22)]   # second is smaller: stale scratch
    for N, M, slices, alpha, beta, seed in cases:
        A = I.normal_bf16(N, M, seed)
        Cin = I.random_c(N, seed + 100, B.DTYPE_BF16_F32)
        want = regular(A, Cin, alpha, beta, slices)
        got = static(A, Cin, alpha, beta, slices)
        _, bound = O.syrk_lower(A, None, alpha, 0.0, B.DTYPE_BF16_F32)
        il, iu = np.tril_indices(N), np.triu_indices(N, 1)
        tol = O.tolerance(M, bound[il], np.abs(Cin[il].astype(np.float64)), alpha, beta, B.DTYPE_BF16_F32)
        err = np.abs(got[il].astype(np.float64) - want[il].astype(np.float64))
        assert np.all(err <= tol), "%d entries differ beyond tolerance" % int((err > tol).sum())
        assert np.array_equal(got[iu], Cin[iu])                      # upper triangle untouched


def test_static_entry_point_refuses_what_does_not_fit():
    N, M = 4096, 512                                                  # 528 tiles x 2 slices > 512
    dA = torch.zeros((N, M), dtype=torch.bfloat16, device="cuda")
    dC = torch.zeros((N, N), dtype=torch.float32, device="cuda")
    with pytest.raises(B.SyrkError) as e:
        B.syrk_lower_bf16_static(N, M, dA, M, dC, N, 1.0, 0.0, 2)
    assert e.value.code == -10
    with pytest.raises(B.SyrkError):
        B.syrk_lower_bf16_static(256, 512, dA, M, dC, N, 1.0, 0.0, 1)        # fewer than 2 slices
