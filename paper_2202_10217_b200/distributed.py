"""K-sharded symmetric rank-k update over several GPUs, one process per GPU (torch.distributed).

The sum over k in Algorithm 1 of the paper splits over blocks of columns of A: with rank r holding the
columns [k_r, k_{r+1}) of A,

    alpha * A A^T + beta * C  =  sum_r (alpha * A_r A_r^T)  +  beta * C .

Every rank runs the library's single-GPU update on its block (triangle blocks, the paper's schedule), the
lower triangles travel in packed form (N (N + 1) / 2 elements instead of N^2), one reduce-scatter sums them
and leaves rank r with a contiguous share of the packed triangle, to which it adds beta times its share of
C.  The paper gives no parallel algorithm (it names them as future work); this is the split that needs a
single collective.  The exchange is torch.distributed's reduce_scatter_tensor (NCCL between GPUs); no
kernel here reads another GPU's memory.

This module only does plumbing: where the columns and the packed entries are cut, buffers, and the order of
the calls.  The arithmetic is in the library's kernels (``binding``) and in the collective.
"""
from __future__ import annotations

from typing import Callable, Optional, Tuple

from . import binding as B

ELEM_BYTES_A = {B.DTYPE_F64: 8, B.DTYPE_BF16_F32: 2, B.DTYPE_TF32_F32: 4, B.DTYPE_E4M3_F32: 1, B.DTYPE_F16_F32: 2}


def column_block(M: int, world: int, rank: int, dtype: int) -> Tuple[int, int]:
    """Columns [k0, k1) of A that `rank` of `world` holds: contiguous blocks of nearly equal width whose
    first column is a multiple of one pipeline stage of the kernels (128 bytes of a row), so that every
    block starts on a 16-byte boundary and no stage straddles two ranks."""
    if world < 1 or not 0 <= rank < world or M < 0:
        raise ValueError("bad world / rank / M")
    step = 128 // ELEM_BYTES_A[dtype]
    steps = (M + step - 1) // step
    lo = (steps * rank) // world * step
    hi = (steps * (rank + 1)) // world * step
    return min(lo, M), min(hi, M)


def packed_share(N: int, world: int, rank: int) -> Tuple[int, int, int]:
    """(first, count, chunk): the packed entries [first, first + count) of the lower triangle that `rank`
    owns after the reduce-scatter; `chunk` is the per-rank length of the exchanged buffer (the packed
    triangle padded with zeros to world * chunk elements, chunk a multiple of 32 elements)."""
    if world < 1 or not 0 <= rank < world or N < 0:
        raise ValueError("bad world / rank / N")
    total = N * (N + 1) // 2
    chunk = ((total + world - 1) // world + 31) // 32 * 32
    first = min(total, rank * chunk)
    return first, min(total, first + chunk) - first, chunk


def exchange_packed(packed_partial, group=None):
    """Sum the ranks' packed partial triangles (each world * chunk elements) and return this rank's chunk."""
    import torch
    import torch.distributed as dist
    world = dist.get_world_size(group)
    if packed_partial.numel() % world != 0:
        raise ValueError("buffer length is not a multiple of the world size")
    out = torch.empty(packed_partial.numel() // world, dtype=packed_partial.dtype, device=packed_partial.device)
    dist.reduce_scatter_tensor(out, packed_partial, op=dist.ReduceOp.SUM, group=group)
    return out


def syrk_lower_ksharded(N: int, M_local: int, A_local, lda: int, C, ldc: int, alpha: float, beta: float, dtype: int,
                        group=None, workspace=None):
    """C_owned <- alpha * sum over ranks of A_r A_r^T + beta * C_owned on this rank's share of the packed lower
    triangle (``packed_share``); every other entry of this rank's C is left as it was.

    `A_local` is this rank's N x M_local block of columns (device tensor, row pitch lda), `C` its N x N
    device tensor (row pitch ldc).  All ranks of `group` call with the same N, alpha, beta and dtype.
    Returns (first, count): the packed range this rank now holds.  `workspace`: optional tuple
    (N x N tensor, packed tensor of world * chunk elements) to reuse between calls.
    """
    import torch
    import torch.distributed as dist
    world, rank = dist.get_world_size(group), dist.get_rank(group)
    first, count, chunk = packed_share(N, world, rank)
    cdt = torch.float64 if dtype == B.DTYPE_F64 else torch.float32
    if workspace is None:
        workspace = (torch.empty((N, N), dtype=cdt, device=C.device),
                     torch.zeros(world * chunk, dtype=cdt, device=C.device))
    W, P = workspace
    if P.numel() != world * chunk or W.shape != (N, N):
        raise ValueError("workspace of the wrong size")
    # 1. this rank's term, scaled: W_lower = alpha * A_r A_r^T (an empty block of columns gives zeros)
    B.syrk_lower(N, M_local, A_local, lda, W, N, alpha, 0.0, dtype)
    # 2. packed form (the padding beyond N (N + 1) / 2 stays zero)
    B.syrk_pack_lower(N, W, N, dtype, P)
    # 3. one collective: sum over ranks, rank r keeps chunk r
    Q = exchange_packed(P, group)
    # 4. C_owned = sum + beta * C_owned
    B.syrk_unpack_lower_axpby(N, first, count, Q, beta, C, ldc, dtype)
    return first, count
