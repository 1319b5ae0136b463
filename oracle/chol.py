"""ctypes front end of the plain-C Cholesky reference (``chol_oracle.c``, Algorithm 2 of the paper).

TEST INFRASTRUCTURE ONLY: imported by the tests and the smoke check, never by the GPU library.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "chol_oracle.c")
_LIB = os.path.join(_HERE, "libchol_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.run(["gcc", "-O2", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared", "-std=c11",
                        "-Wall", "-Wextra", "-o", _LIB, _SRC, "-lm"], check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.oracle_cholesky_lower.restype = ctypes.c_int64
        lib.oracle_cholesky_lower.argtypes = [ctypes.c_int64, ctypes.c_void_p, ctypes.c_int64]
        lib.oracle_cholesky_lower_leading.restype = ctypes.c_int64
        lib.oracle_cholesky_lower_leading.argtypes = [ctypes.c_int64, ctypes.c_int64, ctypes.c_void_p, ctypes.c_int64]
        _lib = lib
    return _lib


def cholesky_lower(A: np.ndarray):
    """Factor of the symmetric positive definite matrix whose lower triangle is in ``A``.

    Returns ``(L, info)``: a copy of ``A`` whose lower triangle holds L (the strict upper
    triangle is left as given) and info = 0, or k + 1 when pivot k is not positive.
    """
    if A.dtype != np.float64 or A.ndim != 2 or A.shape[0] != A.shape[1]:
        raise ValueError("A must be a square float64 array")
    L = np.ascontiguousarray(A).copy()
    info = int(_load().oracle_cholesky_lower(L.shape[0], L.ctypes.data, max(L.shape[0], 1)))
    if info < 0:
        raise ValueError("oracle_cholesky_lower rejected its arguments")
    return L, info


def cholesky_lower_leading(panel: np.ndarray):
    """First ``c`` columns of the factor from the first ``c`` columns of the matrix.

    ``panel`` is N x c (the leading columns of a symmetric positive definite N x N matrix; entries
    above the diagonal are ignored).  Returns ``(Lc, info)`` with the N x c leading columns of L.
    """
    if panel.dtype != np.float64 or panel.ndim != 2 or panel.shape[1] > panel.shape[0]:
        raise ValueError("panel must be a float64 N x c array with c <= N")
    L = np.ascontiguousarray(panel).copy()
    N, c = L.shape
    info = int(_load().oracle_cholesky_lower_leading(N, c, L.ctypes.data, max(c, 1)))
    if info < 0:
        raise ValueError("oracle_cholesky_lower_leading rejected its arguments")
    return L, info


# Parity tolerance of a computed factor against the reference, entry by entry:
#     |L_gpu - L_ref|_ij <= TOL_FACTOR * N * 2^-53 * (|L||L|^T)_ii^(1/2) (|L||L|^T)_jj^(1/2) / L_jj
# is awkward to state; the tests use the standard backward-error form instead:
#     |A - L L^T|_ij <= RESIDUAL_FACTOR * (N + 1) * 2^-53 * (|L||L|^T)_ij .
RESIDUAL_FACTOR = 4.0


def residual_ok(A: np.ndarray, L: np.ndarray):
    """Backward-error check of a computed lower factor (strict upper triangle of L ignored)."""
    N = A.shape[0]
    Ll = np.tril(L)
    R = np.abs(np.tril(A) - np.tril(Ll @ Ll.T))
    bound = RESIDUAL_FACTOR * (N + 1) * 2.0 ** -53 * np.tril(np.abs(Ll) @ np.abs(Ll).T)
    worst = float(np.max(np.where(bound > 0, R / np.maximum(bound, 1e-300), 0.0))) if N else 0.0
    return bool(np.all(R <= bound)), worst
