"""Helpers of the GPU parity tests: run one SYRK call through the C ABI on device
buffers with canaries, and compare it entry by entry with the CPU reference."""
from __future__ import annotations

import numpy as np
import torch

from oracle import syrk as O
from paper_2202_10217_b200 import binding as B
from paper_2202_10217_b200 import inputs as I

GUARD = 3            # canary rows before and after C
SENTINEL = {np.dtype(np.float64): 0x7FF8DEADBEEF1234, np.dtype(np.float32): 0x7FC0BEEF}


def a_to_device(A: np.ndarray, dtype: int, lda: int | None = None, offset_elems: int = 0):
    """Upload A (float64, uint16 bf16 or binary16 bits, float32 for TF32, or uint8 FP8 bytes) with row pitch lda; returns
    (tensor_keepalive, ptr)."""
    N, M = A.shape
    lda = max(M, 1) if lda is None else lda
    tdt = {B.DTYPE_F64: torch.float64, B.DTYPE_BF16_F32: torch.bfloat16, B.DTYPE_TF32_F32: torch.float32,
           B.DTYPE_E4M3_F32: torch.uint8, B.DTYPE_F16_F32: torch.float16}[dtype]
    buf = torch.zeros(offset_elems + max(N, 1) * lda, dtype=tdt, device="cuda")
    if N and M:
        two_byte = dtype in (B.DTYPE_BF16_F32, B.DTYPE_F16_F32)           # uint16 bit patterns
        host = torch.from_numpy(np.ascontiguousarray(A).view(np.int16) if two_byte else np.ascontiguousarray(A))
        if two_byte:
            host = host.view(tdt)
        view = buf[offset_elems:offset_elems + N * lda].view(N, lda)
        view[:, :M].copy_(host)
    return buf, buf.data_ptr() + offset_elems * buf.element_size()


def sentinel_array(shape, np_dtype):
    bits = SENTINEL[np.dtype(np_dtype)]
    u = np.uint64 if np_dtype == np.float64 else np.uint32
    return np.full(shape, bits, dtype=u).view(np_dtype)


def run_case(A: np.ndarray, dtype: int, alpha: float, beta: float, Cin: np.ndarray | None = None,
             lda: int | None = None, ldc: int | None = None, a_offset: int = 0, c_offset: int = 0,
             poison: bool = False, tn: bool = False, upper: bool = False):
    """One call; returns (got, ref, bound).  Checks canaries and status itself.

    `A` is always the N x M operand of the reference.  With `tn` it is handed to the library
    transposed (an M x N row-major array, pitch lda >= N) through syrk_lower_tn.  With `upper`
    the call goes through syrk_ex with the upper triangle stored: the prior values and the result
    live at the mirrored positions (j, i), and `got` is returned transposed so that its lower
    triangle compares with the reference as usual."""
    N, M = A.shape
    cdt = I.c_storage_dtype(dtype)
    ldc = max(N, 1) if ldc is None else ldc
    rows = N + 2 * GUARD
    host_c = sentinel_array((rows, ldc + c_offset), cdt)
    body = host_c[GUARD:GUARD + N, c_offset:c_offset + N] if N else host_c[0:0, 0:0]
    stored = np.tril_indices(N)
    if upper:
        stored = (stored[1], stored[0])                      # entry (i, j), j <= i, lives at (j, i)
    if Cin is not None:
        body[stored] = Cin[np.tril_indices(N)]
    elif poison:
        body[stored] = np.nan
    before = host_c.copy()
    dev_c = torch.from_numpy(host_c).cuda()
    c_ptr = dev_c.data_ptr() + (GUARD * (ldc + c_offset) + c_offset) * dev_c.element_size()
    if tn:
        keep, a_ptr = a_to_device(np.ascontiguousarray(A.T), dtype, lda, a_offset)
        lda_eff = max(N, 1) if lda is None else lda
    else:
        keep, a_ptr = a_to_device(A, dtype, lda, a_offset)
        lda_eff = max(M, 1) if lda is None else lda
    if upper:
        B.syrk_ex(B.UPLO_UPPER, B.OP_T if tn else B.OP_N, N, M, a_ptr, lda_eff, c_ptr, ldc + c_offset, alpha, beta, dtype)
    elif tn:
        B.syrk_lower_tn(N, M, a_ptr, lda_eff, c_ptr, ldc + c_offset, alpha, beta, dtype)
    else:
        B.syrk_lower(N, M, a_ptr, lda_eff, c_ptr, ldc + c_offset, alpha, beta, dtype)
    torch.cuda.synchronize()
    assert B.syrk_last_status() == 0
    after = dev_c.cpu().numpy()
    u = np.uint64 if cdt == np.float64 else np.uint32
    # everything outside the lower triangle is bitwise untouched
    mask = np.ones(after.shape, dtype=bool)
    if N:
        m = mask[GUARD:GUARD + N, c_offset:c_offset + N]
        m[stored] = False
    assert np.array_equal(after.view(u)[mask], before.view(u)[mask]), "wrote outside the stored triangle"
    got = after[GUARD:GUARD + N, c_offset:c_offset + N].astype(np.float64)
    if upper:
        got = np.ascontiguousarray(got.T)
    ref, bound = O.syrk_lower(np.ascontiguousarray(A), None if Cin is None else np.ascontiguousarray(Cin),
                              alpha, beta if Cin is not None else 0.0, dtype)
    return got, ref, bound


def assert_within_tolerance(got, ref, bound, M, alpha, beta, Cin, dtype, exact=False):
    N = got.shape[0]
    il = np.tril_indices(N)
    g, r = got[il], ref[il]
    assert not np.isnan(g).any()
    if exact:
        assert np.array_equal(g, r), "max abs diff %g" % np.max(np.abs(g - r))
        return 0.0
    tol = O.tolerance(M, bound[il], None if Cin is None else np.abs(Cin[il].astype(np.float64)),
                      alpha, beta, dtype)
    err = np.abs(g - r)
    bad = err > tol
    assert not bad.any(), "%d entries out of tolerance, worst ratio %g" % (
        int(bad.sum()), float(np.max(err[bad] / np.maximum(tol[bad], 1e-300))))
    with np.errstate(divide="ignore", invalid="ignore"):
        ratio = np.where(tol > 0, err / tol, 0.0)
    return float(ratio.max()) if ratio.size else 0.0
