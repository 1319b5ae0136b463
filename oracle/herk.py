"""ctypes front end of the plain-C Hermitian rank-k reference (``herk_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, never by the GPU library or its binding.
The arithmetic lives in the C file; this module compiles it with gcc and marshals numpy arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "herk_oracle.c")
_LIB = os.path.join(_HERE, "libherk_oracle.so")

# Parity tolerance, per part (real, imaginary) of an entry:
#   |part_gpu - part_ref| <= TOL * 2M * (|alpha| Bound_part + |beta| |C_in part|)
# - each part is a sum of 2M real products, so this is the rank-k update's tolerance with 2M terms.
TOL = 8.0 * 2.0 ** -53


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
        lib.oracle_herk_lower.restype = ctypes.c_int
        lib.oracle_herk_lower.argtypes = [i64, i64, vp, i64, vp, i64, dbl, dbl, vp, vp, i64]
        _lib = lib
    return _lib


def herk_lower(A: np.ndarray, C_in, alpha: float, beta: float):
    """Reference lower triangle of alpha A A^H + beta C (complex128) and the bound, as a complex array whose
    real part bounds the real part's products and whose imaginary part the imaginary part's.
    Returns (C_ref, Bound): N x N complex arrays whose strict upper triangles are NaN (never written)."""
    if A.dtype != np.complex128 or A.ndim != 2 or (A.size > 0 and A.strides[1] != 16):
        raise ValueError("A must be a row-major 2-D complex128 array")
    N, M = A.shape
    ref = np.full((N, N), complex(np.nan, np.nan))
    bound = np.full((N, N), complex(np.nan, np.nan))
    cptr, ldc = None, max(N, 1)
    if C_in is not None:
        if C_in.dtype != np.complex128 or C_in.strides[1] != 16:
            raise ValueError("C must be a row-major complex128 array")
        cptr, ldc = C_in.ctypes.data, C_in.strides[0] // 16
    lda = max(A.strides[0] // 16, M, 1) if A.size else max(M, 1)
    rc = _load().oracle_herk_lower(N, M, A.ctypes.data, lda, cptr, ldc, float(alpha), float(beta),
                                   ref.ctypes.data, bound.ctypes.data, max(N, 1))
    if rc != 0:
        raise ValueError("oracle_herk_lower rejected its arguments")
    return ref, bound


def tolerance(M: int, bound: np.ndarray, c_in, alpha: float, beta: float) -> np.ndarray:
    """Per-part tolerance as a complex array (real part: tolerance of the real part, and likewise)."""
    tr = abs(alpha) * bound.real
    ti = abs(alpha) * bound.imag
    if c_in is not None and beta != 0.0:
        tr = tr + abs(beta) * np.abs(c_in.real)
        ti = ti + abs(beta) * np.abs(c_in.imag)
    scale = TOL * 2.0 * max(M, 1)
    return scale * tr + 1j * (scale * ti)
