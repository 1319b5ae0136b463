"""The allocation-free K-split entry point against the CPU reference and the regular entry point.

syrk_lower_bf16_static is for callers that cannot let the library call cudaMalloc; it
keeps its work list and partial tiles in fixed device arrays.  Its result must agree
with the CPU reference within the BF16 parity tolerance and with syrk_lower (triangle
blocks, same K-split: the same sums in the same order) bit for bit, on calls in a row
with different problems (a later call reuses the arrays an earlier one wrote; the third
repeats the second's size, for which the work list is not uploaded again).  Its own
status word must stay clear.  Collected last, so that a failure here cannot hide another
test's result.
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
        B.syrk_set_schedule(B.SCHEDULE_TBS)            # the static entry point runs the triangle-block kernel
        B.syrk_set_split_k(slices)
        B.syrk_lower(N, M, dA, M, dC, N, alpha, beta, B.DTYPE_BF16_F32)
        torch.cuda.synchronize()
    finally:
        B.syrk_set_split_k(0)
        B.syrk_set_schedule(B.SCHEDULE_DEFAULT)
    assert B.syrk_last_status() == 0
    return dC.cpu().numpy()


def static(A, Cin, alpha, beta, slices):
    N, M = A.shape
    dA = torch.from_numpy(A.view(np.int16)).cuda().view(torch.bfloat16)
    dC = torch.from_numpy(Cin.copy()).cuda()
    B.syrk_lower_bf16_static(N, M, dA, M, dC, N, alpha, beta, slices)
    torch.cuda.synchronize()
    assert B.syrk_lower_bf16_static_status() == 0
    return dC.cpu().numpy()


def test_static_entry_point_matches_reference_and_regular_one_on_calls_in_a_row():
    cases = [(1500, 2048, 4, 1.0, 0.0, 21), (900, 1280, 6, -1.0, 1.0, 22),   # second is smaller: stale scratch
             (900, 640, 3, 0.5, 2.0, 23)]                                     # same size again: cached work list
    for N, M, slices, alpha, beta, seed in cases:
        A = I.normal_bf16(N, M, seed)
        Cin = I.random_c(N, seed + 100, B.DTYPE_BF16_F32)
        got = static(A, Cin, alpha, beta, slices)
        ref, bound = O.syrk_lower(A, Cin, alpha, beta, B.DTYPE_BF16_F32)
        il, iu = np.tril_indices(N), np.triu_indices(N, 1)
        tol = O.tolerance(M, bound[il], np.abs(Cin[il].astype(np.float64)), alpha, beta, B.DTYPE_BF16_F32)
        err = np.abs(got[il].astype(np.float64) - ref[il])
        assert np.all(err <= tol), "%d entries beyond tolerance of the reference" % int((err > tol).sum())
        assert np.array_equal(got[iu], Cin[iu])                      # upper triangle untouched
        want = regular(A, Cin, alpha, beta, slices)
        assert np.array_equal(got[il], want[il])                     # same slices summed in the same order


def test_static_entry_point_refuses_a_stream_under_capture():
    N, M = 512, 1024
    dA = torch.zeros((N, M), dtype=torch.bfloat16, device="cuda")
    dC = torch.zeros((N, N), dtype=torch.float32, device="cuda")
    B.syrk_lower_bf16_static(N, M, dA, M, dC, N, 1.0, 0.0, 2)            # first call on the device: outside capture
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        dC.mul_(1.0)
        with pytest.raises(B.SyrkError) as e:
            B.syrk_lower_bf16_static(N, M, dA, M, dC, N, 1.0, 0.0, 2, stream=side.cuda_stream)
        assert e.value.code == -6
    torch.cuda.synchronize()
    assert B.syrk_lower_bf16_static_status() == 0


def test_static_entry_point_refuses_what_does_not_fit():
    N, M = 4096, 512                                                  # 528 tiles x 2 slices > 512
    dA = torch.zeros((N, M), dtype=torch.bfloat16, device="cuda")
    dC = torch.zeros((N, N), dtype=torch.float32, device="cuda")
    with pytest.raises(B.SyrkError) as e:
        B.syrk_lower_bf16_static(N, M, dA, M, dC, N, 1.0, 0.0, 2)
    assert e.value.code == -10
    with pytest.raises(B.SyrkError):
        B.syrk_lower_bf16_static(256, 512, dA, M, dC, N, 1.0, 0.0, 1)        # fewer than 2 slices
