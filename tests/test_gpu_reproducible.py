"""Run-to-run bitwise reproducibility on the GPU: every path that sums partial results (K-splits of both
kernels), the persistent launch forms (items drawn from a counter), the batch and the rank-2k update must
give the same bits when the same call is repeated - a race between blocks or a data-dependent summation
order would show up here."""
import numpy as np
import pytest
import torch

from paper_2202_10217_b200 import binding as B
from paper_2202_10217_b200 import inputs as I

from gpu_util import a_to_device
from test_gpu_syrk import BOTH, make_A

pytestmark = pytest.mark.gpu
DT = pytest.mark.parametrize("dtype", BOTH, ids=["f64", "bf16", "tf32", "e4m3", "f16"])


def repeat(call, dC, fill, times=4):
    outs = []
    for _ in range(times):
        dC.copy_(fill)
        call()
        torch.cuda.synchronize()
        assert B.syrk_last_status() == 0
        outs.append(dC.clone())
    for o in outs[1:]:
        assert torch.equal(o.view(torch.uint8), outs[0].view(torch.uint8))     # bit for bit (NaN-safe)


@DT
@pytest.mark.parametrize("split", [0, 3, 8])
def test_repeated_calls_give_the_same_bits(dtype, split):
    N, M = (1500, 2100) if dtype == B.DTYPE_F64 else (1408, 4096)
    A = make_A(N, M, dtype, seed=6000)
    keep, a_ptr = a_to_device(A, dtype)
    cdt = torch.float64 if dtype == B.DTYPE_F64 else torch.float32
    fill = torch.randn((N, N), dtype=cdt, device="cuda", generator=torch.Generator(device="cuda").manual_seed(1))
    dC = torch.empty_like(fill)
    try:
        B.syrk_set_split_k(split)
        repeat(lambda: B.syrk_lower(N, M, a_ptr, M, dC, N, 1.5, -0.5, dtype), dC, fill)
        repeat(lambda: B.syrk_ex(B.UPLO_UPPER, B.OP_N, N, M, a_ptr, M, dC, N, 1.5, -0.5, dtype), dC, fill)
    finally:
        B.syrk_set_split_k(0)


def test_f64_persistent_form_batch_and_rank_2k_update():
    N, M = 4500, 256
    A = torch.from_numpy(I.normal_f64(N, M, 6100)).cuda()
    Bm = torch.from_numpy(I.normal_f64(N, M, 6101)).cuda()
    fill = torch.randn((N, N), dtype=torch.float64, device="cuda", generator=torch.Generator(device="cuda").manual_seed(2))
    dC = torch.empty_like(fill)
    try:
        B.syrk_set_f64_launch(B.F64_LAUNCH_PERSISTENT)
        repeat(lambda: B.syrk_lower(N, M, A, M, dC, N, -1.0, 1.0, B.DTYPE_F64), dC, fill)
    finally:
        B.syrk_set_f64_launch(B.F64_LAUNCH_AUTO)
    repeat(lambda: B.syr2k_lower(N, M, A, M, Bm, M, dC, N, -1.0, 1.0), dC, fill)
    nb, n = 9, 500
    repeat(lambda: B.syrk_lower_batched(nb, n, M, A, M, n * M, dC, n, n * n, 1.0, 0.5, B.DTYPE_F64), dC, fill)
