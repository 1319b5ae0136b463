"""ctypes front end of the plain-C SYRK reference (``syrk_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the
CPU-baseline leg of the benchmark, never by the GPU library or its binding.

The arithmetic lives in the C file (Algorithm 1 of the paper plus alpha/beta);
this module only compiles it with gcc and marshals numpy arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "syrk_oracle.c")
_LIB = os.path.join(_HERE, "libsyrk_oracle.so")

DTYPE_F64 = 0
DTYPE_BF16_F32 = 1
DTYPE_TF32_F32 = 2
DTYPE_E4M3_F32 = 3
DTYPE_F16_F32 = 4


def build(force: bool = False) -> str:
    """Compile the C reference into a shared object next to its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared",
               "-std=c11", "-Wall", "-Wextra", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i64, dbl, vp = ctypes.c_int64, ctypes.c_double, ctypes.c_void_p
        lib.oracle_syrk_lower.restype = ctypes.c_int
        lib.oracle_syrk_lower.argtypes = [i64, i64, vp, i64, vp, i64, dbl, dbl,
                                          ctypes.c_int, vp, vp, i64]
        lib.oracle_syrk_entries.restype = ctypes.c_int
        lib.oracle_syrk_entries.argtypes = [i64, vp, vp, i64, i64, vp, i64, vp, i64,
                                            dbl, dbl, ctypes.c_int, vp, vp]
        lib.oracle_num_threads.restype = ctypes.c_int
        lib.oracle_widen.restype = ctypes.c_int
        lib.oracle_widen.argtypes = [i64, i64, vp, i64, ctypes.c_int, vp]
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def _check_inputs(A: np.ndarray, C_in, dtype: int):
    want_a = {DTYPE_F64: np.float64, DTYPE_BF16_F32: np.uint16, DTYPE_TF32_F32: np.float32,
              DTYPE_E4M3_F32: np.uint8, DTYPE_F16_F32: np.uint16}[dtype]
    want_c = np.float64 if dtype == DTYPE_F64 else np.float32
    if A.dtype != want_a or A.ndim != 2 or (A.size > 0 and A.strides[1] != A.itemsize):
        raise ValueError("A must be a row-major 2-D array of %s" % want_a.__name__)
    if C_in is not None and (C_in.dtype != want_c or C_in.ndim != 2
                             or C_in.strides[1] != C_in.itemsize):
        raise ValueError("C must be a row-major 2-D array of %s" % want_c.__name__)


def widen(A: np.ndarray, dtype: int) -> np.ndarray:
    """The operand as binary64 values, every element decoded exactly from its storage format (bf16 or
    binary16 bit patterns, binary32 read as TF32, FP8 E4M3 bytes) by the reference's own decoder."""
    _check_inputs(A, None, dtype)
    N, M = A.shape
    out = np.empty((N, M), dtype=np.float64)
    lda = max(A.strides[0] // A.itemsize, M, 1) if A.size > 0 else max(M, 1)
    if _load().oracle_widen(N, M, A.ctypes.data, lda, dtype, out.ctypes.data) != 0:
        raise ValueError("oracle_widen rejected its arguments")
    return out


def syrk_lower(A: np.ndarray, C_in, alpha: float, beta: float, dtype: int):
    """Reference lower triangle and bound matrix.

    ``A`` is N x M (float64, uint16 holding bf16 bit patterns, or float32 read as TF32:
    its 13 low-order bits are dropped, or uint8 holding FP8 E4M3 bytes, or uint16 holding
    binary16 bit patterns for ``DTYPE_F16_F32``); ``C_in`` is the
    N x N prior value (float64 / float32) or None when beta == 0.  Returns
    ``(C_ref, B)``: N x N float64 arrays whose strict upper triangles are NaN
    (never written), with ``B[i, j] = sum_k |A[i,k]| |A[j,k]|``.
    """
    _check_inputs(A, C_in, dtype)
    N, M = A.shape
    lda = max(A.strides[0] // A.itemsize, M, 1) if A.size > 0 else max(M, 1)
    ref = np.full((N, N), np.nan, dtype=np.float64)
    bound = np.full((N, N), np.nan, dtype=np.float64)
    cptr, ldc = None, max(N, 1)
    if C_in is not None:
        cptr, ldc = C_in.ctypes.data, C_in.strides[0] // C_in.itemsize
    rc = _load().oracle_syrk_lower(N, M, A.ctypes.data, lda, cptr, ldc, float(alpha),
                                   float(beta), dtype, ref.ctypes.data, bound.ctypes.data,
                                   max(N, 1))
    if rc != 0:
        raise ValueError("oracle_syrk_lower rejected its arguments")
    return ref, bound


def syrk_entries(I, J, A: np.ndarray, C_in, alpha: float, beta: float, dtype: int):
    """Reference values and bounds of the listed entries (I[p] >= J[p])."""
    _check_inputs(A, C_in, dtype)
    I = np.ascontiguousarray(I, dtype=np.int64)
    J = np.ascontiguousarray(J, dtype=np.int64)
    N, M = A.shape
    lda = A.strides[0] // A.itemsize
    ref = np.empty(I.shape[0], dtype=np.float64)
    bound = np.empty(I.shape[0], dtype=np.float64)
    cptr, ldc = None, max(N, 1)
    if C_in is not None:
        cptr, ldc = C_in.ctypes.data, C_in.strides[0] // C_in.itemsize
    rc = _load().oracle_syrk_entries(I.shape[0], I.ctypes.data, J.ctypes.data, N, M,
                                     A.ctypes.data, lda, cptr, ldc, float(alpha),
                                     float(beta), dtype, ref.ctypes.data, bound.ctypes.data)
    if rc != 0:
        raise ValueError("oracle_syrk_entries rejected its arguments")
    return ref, bound


# Parity tolerance: |C_gpu - C_ref| <= TOL[dtype] * M * (|alpha| B + |beta| |C_in|).
TOL = {DTYPE_F64: 8.0 * 2.0 ** -53, DTYPE_BF16_F32: 4.0 * 2.0 ** -24, DTYPE_TF32_F32: 4.0 * 2.0 ** -24,
       DTYPE_E4M3_F32: 4.0 * 2.0 ** -24, DTYPE_F16_F32: 4.0 * 2.0 ** -24}


def tolerance(M: int, bound, c_in_abs, alpha: float, beta: float, dtype: int):
    """Per-entry allowed deviation (same shape as ``bound``)."""
    t = abs(alpha) * np.asarray(bound, dtype=np.float64)
    if beta != 0.0 and c_in_abs is not None:
        t = t + abs(beta) * np.asarray(c_in_abs, dtype=np.float64)
    return TOL[dtype] * max(int(M), 1) * t
