"""Host logic of the K-sharded multi-GPU update on CPU: where the columns of A and the packed entries of
the triangle are cut, and the exchange itself with two gloo ranks.

Each rank computes its own term alpha * A_r A_r^T with the CPU reference (standing in for the GPU kernel,
which the GPU tests check), packs its lower triangle, and the ranks sum the packed triangles with the same
reduce-scatter call the GPU path uses; the owned shares, put together, must equal the reference result for
the whole A (integer inputs: bit for bit)."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2202_10217_b200 import binding as B
from paper_2202_10217_b200 import distributed as D
from paper_2202_10217_b200 import inputs as I


def test_column_blocks_tile_the_inner_dimension_on_stage_boundaries():
    for dtype, step in ((B.DTYPE_F64, 16), (B.DTYPE_BF16_F32, 64), (B.DTYPE_TF32_F32, 32), (B.DTYPE_E4M3_F32, 128)):
        for M in (0, 1, 63, 64, 1000, 4096, 262144):
            for world in (1, 2, 3, 8):
                blocks = [D.column_block(M, world, r, dtype) for r in range(world)]
                assert blocks[0][0] == 0 and blocks[-1][1] == M
                for (a0, a1), (b0, b1) in zip(blocks, blocks[1:]):
                    assert a1 == b0 and a0 <= a1
                assert all(k0 % step == 0 for k0, _ in blocks)
                widths = [k1 - k0 for k0, k1 in blocks]
                assert max(widths) - min(widths) <= 2 * step          # nearly equal shares
    with pytest.raises(ValueError):
        D.column_block(10, 2, 2, B.DTYPE_F64)


def test_packed_shares_tile_the_triangle():
    for N in (0, 1, 5, 127, 1000):
        total = N * (N + 1) // 2
        for world in (1, 2, 3, 8):
            shares = [D.packed_share(N, world, r) for r in range(world)]
            chunk = shares[0][2]
            assert chunk % 32 == 0 and world * chunk >= total
            covered = 0
            for first, count, ch in shares:
                assert ch == chunk and first == min(total, covered) and count >= 0
                covered = first + count
            assert covered == total


def _rank_main(rank, world, port, out, N, M, dtype, alpha, beta):
    from oracle import syrk as O
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    A = I.small_int_f64(N, M, 5) if dtype == B.DTYPE_F64 else I.small_int_bf16(N, M, 5)
    Cin = np.round(I.random_c(N, 6, dtype) * 4).astype(I.c_storage_dtype(dtype))
    k0, k1 = D.column_block(M, world, rank, dtype)
    first, count, chunk = D.packed_share(N, world, rank)
    il = np.tril_indices(N)
    if k1 > k0:
        W, _ = O.syrk_lower(np.ascontiguousarray(A[:, k0:k1]), None, alpha, 0.0, dtype)     # this rank's term
    else:
        W = np.zeros((N, N))
    packed = np.zeros(world * chunk, dtype=I.c_storage_dtype(dtype))
    packed[:il[0].size] = W[il].astype(packed.dtype)          # tril_indices runs row by row: the packed order
    mine = D.exchange_packed(torch.from_numpy(packed)).numpy()
    own = mine[:count].astype(np.float64) + beta * Cin[il][first:first + count].astype(np.float64)
    out.put((rank, first, count, own))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("dtype,N,M", [(B.DTYPE_F64, 150, 70), (B.DTYPE_BF16_F32, 97, 200), (B.DTYPE_F64, 40, 10)])
def test_two_ranks_reduce_scatter_gives_the_reference_result(dtype, N, M):
    from oracle import syrk as O
    alpha, beta = 2.0, -1.0
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29700 + (os.getpid() + N) % 1500
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out, N, M, dtype, alpha, beta)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    A = I.small_int_f64(N, M, 5) if dtype == B.DTYPE_F64 else I.small_int_bf16(N, M, 5)
    Cin = np.round(I.random_c(N, 6, dtype) * 4).astype(I.c_storage_dtype(dtype))
    ref, _ = O.syrk_lower(A, Cin, alpha, beta, dtype)
    il = np.tril_indices(N)
    whole = np.concatenate([g[3] for g in got])
    assert [g[1] for g in got] == [0, got[0][2]] and whole.size == il[0].size      # shares are adjacent and complete
    assert np.array_equal(whole, ref[il])                                           # integers: exact in any order
