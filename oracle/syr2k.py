"""ctypes front end of the plain-C rank-2k reference (``syr2k_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, never by the GPU library or its binding.
The arithmetic lives in the C file; this module compiles it with gcc and marshals numpy arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "syr2k_oracle.c")
_LIB = os.path.join(_HERE, "libsyr2k_oracle.so")

# Parity tolerance: |C_gpu - C_ref| <= TOL * 2M * (|alpha| Bd + |beta| |C_in|): 2M products per entry.
TOL = 8.0 * 2.0 ** -53
# ... and for the input types whose products are exact in binary32 and are accumulated in binary32 (bfloat16,
# binary16, TF32, FP8 E4M3): the tolerance of the rank-k update on those types, again with 2M products.
TOL_F32_ACC = 4.0 * 2.0 ** -24


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.run(["gcc", "-O2", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-Wall",
                        "-Wextra", "-o", _LIB, _SRC, "-lm"], check=True)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i64, dbl, vp = ctypes.c_int64, ctypes.c_double, ctypes.c_void_p
        lib.oracle_syr2k_lower.restype = ctypes.c_int
        lib.oracle_syr2k_lower.argtypes = [i64, i64, vp, i64, vp, i64, vp, i64, dbl, dbl, vp, vp, i64]
        _lib = lib
    return _lib


def syr2k_lower(A: np.ndarray, B: np.ndarray, C_in, alpha: float, beta: float):
    """Reference lower triangle and bound matrix of alpha (A B^T + B A^T) + beta C (binary64).
    Returns (C_ref, Bd): N x N arrays whose strict upper triangles are NaN (never written)."""
    for X in (A, B):
        if X.dtype != np.float64 or X.ndim != 2 or (X.size > 0 and X.strides[1] != 8):
            raise ValueError("A and B must be row-major 2-D float64 arrays")
    if A.shape != B.shape:
        raise ValueError("A and B must have the same shape")
    N, M = A.shape
    ref = np.full((N, N), np.nan)
    bound = np.full((N, N), np.nan)
    cptr, ldc = None, max(N, 1)
    if C_in is not None:
        if C_in.dtype != np.float64 or C_in.strides[1] != 8:
            raise ValueError("C must be a row-major float64 array")
        cptr, ldc = C_in.ctypes.data, C_in.strides[0] // 8
    lda = max(A.strides[0] // 8, M, 1) if A.size else max(M, 1)
    ldb = max(B.strides[0] // 8, M, 1) if B.size else max(M, 1)
    rc = _load().oracle_syr2k_lower(N, M, A.ctypes.data, lda, B.ctypes.data, ldb, cptr, ldc, float(alpha),
                                    float(beta), ref.ctypes.data, bound.ctypes.data, max(N, 1))
    if rc != 0:
        raise ValueError("oracle_syr2k_lower rejected its arguments")
    return ref, bound


def syr2k_lower_typed(A: np.ndarray, B: np.ndarray, C_in, alpha: float, beta: float, dtype: int):
    """The same reference for operands in one of the library's storage types (dtype codes of the rank-k
    reference): both operands are decoded exactly to binary64 by that reference's decoder, a binary32 C_in
    is widened exactly, and the binary64 definition above is applied (products of two decoded values have
    at most 22 significant bits, so each product is exact; only the sums round, in binary64)."""
    from . import syrk as _syrk
    if dtype == _syrk.DTYPE_F64:
        return syr2k_lower(A, B, C_in, alpha, beta)
    A64, B64 = _syrk.widen(np.ascontiguousarray(A), dtype), _syrk.widen(np.ascontiguousarray(B), dtype)
    C64 = None
    if C_in is not None:
        if C_in.dtype != np.float32:
            raise ValueError("C must be float32 for this input type")
        C64 = np.ascontiguousarray(C_in, dtype=np.float64)
    return syr2k_lower(A64, B64, C64, alpha, beta)


def tolerance(M: int, bound, c_in_abs, alpha: float, beta: float, f32_accumulate: bool = False):
    t = abs(alpha) * np.asarray(bound, dtype=np.float64)
    if beta != 0.0 and c_in_abs is not None:
        t = t + abs(beta) * np.asarray(c_in_abs, dtype=np.float64)
    return (TOL_F32_ACC if f32_accumulate else TOL) * 2 * max(int(M), 1) * t
