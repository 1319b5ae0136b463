"""The K-sharded update on the GPU: the packed-triangle kernels and the per-rank sequence of calls.

One GPU is available, so (a) the whole path runs with a process group of one rank (NCCL), and (b) the terms
of two and three ranks are computed one after the other on the same GPU - each rank's block of columns
through syrk_lower and syrk_pack_lower - and added with torch in place of the collective's sum; every
rank's share is then put into C by syrk_unpack_lower_axpby.  Both must give the CPU reference's result
(the two-process exchange itself is covered on CPU with gloo)."""
import os

import numpy as np
import pytest
import torch
import torch.distributed as dist

from oracle import syrk as O
from paper_2202_10217_b200 import binding as B
from paper_2202_10217_b200 import distributed as D
from paper_2202_10217_b200 import inputs as I

from test_gpu_configs import upload_A
from test_gpu_syrk import make_A

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,N,M", [(B.DTYPE_F64, 1100, 200), (B.DTYPE_BF16_F32, 1300, 520)])
def test_terms_of_several_ranks_packed_summed_and_unpacked(dtype, N, M):
    for world in (2, 3):
        A = make_A(N, M, dtype, seed=9100 + world, kind="int")
        Cin = np.round(I.random_c(N, 9101, dtype, ldc=N + 3) * 4).astype(I.c_storage_dtype(dtype))
        alpha, beta = -1.0, 2.0
        cdt = torch.float64 if dtype == B.DTYPE_F64 else torch.float32
        dC = torch.from_numpy(Cin.copy()).cuda()
        chunk = D.packed_share(N, world, 0)[2]
        total = torch.zeros(world * chunk, dtype=cdt, device="cuda")
        for r in range(world):
            k0, k1 = D.column_block(M, world, r, dtype)
            dA = upload_A(np.ascontiguousarray(A[:, k0:k1]), dtype) if k1 > k0 else torch.zeros(1, device="cuda")
            W = torch.full((N, N), float("nan"), dtype=cdt, device="cuda")
            P = torch.zeros(world * chunk, dtype=cdt, device="cuda")
            B.syrk_lower(N, k1 - k0, dA, max(k1 - k0, 1), W, N, alpha, 0.0, dtype)
            B.syrk_pack_lower(N, W, N, dtype, P)
            total += P                                              # stands in for the collective's sum
        for r in range(world):
            first, count, _ = D.packed_share(N, world, r)
            B.syrk_unpack_lower_axpby(N, first, count, total[r * chunk:], beta, dC, N + 3, dtype)
        torch.cuda.synchronize()
        assert B.syrk_last_status() == 0
        got = dC.cpu().numpy()
        ref, _ = O.syrk_lower(A, np.ascontiguousarray(Cin[:, :N]), alpha, beta, dtype)
        il, iu = np.tril_indices(N), np.triu_indices(N, 1)
        assert np.array_equal(got[:, :N][il].astype(np.float64), ref[il])          # integers: exact
        assert np.array_equal(got[:, :N][iu], Cin[:, :N][iu]) and np.array_equal(got[:, N:], Cin[:, N:])


def test_whole_path_with_a_process_group_of_one_rank():
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", str(29900 + os.getpid() % 1000))
    created = not dist.is_initialized()
    if created:
        dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", torch.cuda.current_device()))
    try:
        for dtype, N, M in [(B.DTYPE_F64, 900, 130), (B.DTYPE_BF16_F32, 1000, 260)]:
            A = make_A(N, M, dtype, seed=9200)
            Cin = I.random_c(N, 9201, dtype)
            dA = upload_A(A, dtype)
            dC = torch.from_numpy(Cin.copy()).cuda()
            first, count = D.syrk_lower_ksharded(N, M, dA, M, dC, N, 0.5, -1.5, dtype)
            torch.cuda.synchronize()
            assert (first, count) == (0, N * (N + 1) // 2) and B.syrk_last_status() == 0
            ref, bound = O.syrk_lower(A, Cin, 0.5, -1.5, dtype)
            il, iu = np.tril_indices(N), np.triu_indices(N, 1)
            tol = O.tolerance(M, bound[il], np.abs(Cin[il].astype(np.float64)), 0.5, -1.5, dtype)
            got = dC.cpu().numpy()
            assert np.all(np.abs(got[il].astype(np.float64) - ref[il]) <= tol)
            assert np.array_equal(got[iu], Cin[iu])
    finally:
        if created:
            dist.destroy_process_group()


def test_packed_kernels_reject_bad_ranges():
    dC = torch.zeros((8, 8), dtype=torch.float64, device="cuda")
    P = torch.zeros(64, dtype=torch.float64, device="cuda")
    with pytest.raises(B.SyrkError):
        B.syrk_unpack_lower_axpby(8, 30, 10, P, 0.0, dC, 8, B.DTYPE_F64)       # 30 + 10 > 36
    with pytest.raises(B.SyrkError):
        B.syrk_pack_lower(8, dC, 7, B.DTYPE_F64, P)                             # ldc < N
