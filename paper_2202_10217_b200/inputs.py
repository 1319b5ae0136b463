"""Seeded synthetic inputs for the SYRK workloads.

This module only draws random numbers, rounds them to the storage type and
shapes them; it contains none of the method's arithmetic, so both the GPU tests
and the CPU reference may take their inputs from it.  All generators are numpy
``default_rng(seed)`` streams on the host, so the bits do not depend on torch or
on a GPU.

bf16 values travel as ``uint16`` bit patterns and FP8 E4M3 values as ``uint8`` bytes (numpy has
neither type); binary16 values travel as ``uint16`` bit patterns too, so that every 16-bit
input reaches the library the same way.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Optional

import numpy as np

DTYPE_F64 = 0        # A, C binary64
DTYPE_BF16_F32 = 1   # A bfloat16, C binary32 (binary32 accumulation)
DTYPE_TF32_F32 = 2   # A binary32 read as TF32 (19 high-order bits), C binary32
DTYPE_E4M3_F32 = 3   # A FP8 E4M3 bytes (uint8), C binary32
DTYPE_F16_F32 = 4    # A IEEE binary16 bit patterns (uint16), C binary32


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round binary32 values to bfloat16 (nearest, ties to even); returns uint16 bits."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    rounded = (u + np.uint32(0x7FFF) + lsb) >> np.uint32(16)
    return rounded.astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Widen bfloat16 bit patterns to binary32 (exact)."""
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def f32_to_f16_bits(x: np.ndarray) -> np.ndarray:
    """Round binary32 values to IEEE binary16 (nearest, ties to even; numpy's conversion); uint16 bits."""
    return np.ascontiguousarray(x, dtype=np.float32).astype(np.float16).view(np.uint16)


def f16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Widen binary16 bit patterns to binary32 (exact)."""
    return np.ascontiguousarray(bits, dtype=np.uint16).view(np.float16).astype(np.float32)


def f32_keep_tf32_bits(x: np.ndarray) -> np.ndarray:
    """binary32 values with the 13 low-order bits cleared (exactly representable in TF32)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32) & np.uint32(0xFFFFE000)
    return u.view(np.float32)


def e4m3_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Decode FP8 E4M3 bytes (1-4-3, bias 7, no infinities, NaN = 0x7F / 0xFF) to binary32 (exact)."""
    b = np.ascontiguousarray(bits, dtype=np.uint8).astype(np.int32)
    e, f = (b >> 3) & 15, b & 7
    mag = np.where(e == 0, np.ldexp(f.astype(np.float32), -9), np.ldexp((8 + f).astype(np.float32), e - 10))
    mag = np.where((e == 15) & (f == 7), np.float32(np.nan), mag).astype(np.float32)
    return np.where(b >> 7 == 1, -mag, mag).astype(np.float32)


def f32_to_e4m3_bits(x: np.ndarray) -> np.ndarray:
    """Round binary32 values to FP8 E4M3 (nearest, ties to the even code, saturating at +-448)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    grid = e4m3_bits_to_f32(np.arange(0, 127, dtype=np.uint8)).astype(np.float64)     # codes 0..126: 0..448
    a = np.minimum(np.abs(x).astype(np.float64), 448.0)
    hi = np.clip(np.searchsorted(grid, a, side="left"), 0, 126)
    lo = np.maximum(hi - 1, 0)
    d_lo, d_hi = a - grid[lo], grid[hi] - a
    take_lo = (d_lo < d_hi) | ((d_lo == d_hi) & (lo % 2 == 0))
    code = np.where(take_lo, lo, hi).astype(np.uint8)
    return (code | (np.signbit(x).astype(np.uint8) << 7)).astype(np.uint8)


def _normal(rng: np.random.Generator, shape, std: float, chunk_rows: int = 1024) -> np.ndarray:
    """N(0, std^2) float32 array drawn row-chunk by row-chunk (bounded host memory)."""
    out = np.empty(shape, dtype=np.float32)
    for r0 in range(0, shape[0], chunk_rows):
        r1 = min(shape[0], r0 + chunk_rows)
        out[r0:r1] = (rng.standard_normal((r1 - r0, shape[1]), dtype=np.float32) * np.float32(std))
    return out


def uniform_f64(N: int, M: int, seed: int) -> np.ndarray:
    """Entries i.i.d. Uniform(-1, 1), binary64."""
    return np.random.default_rng(seed).uniform(-1.0, 1.0, size=(N, M))


def normal_f64(N: int, M: int, seed: int, std: float = 1.0) -> np.ndarray:
    """Entries i.i.d. N(0, std^2), binary64."""
    return np.random.default_rng(seed).standard_normal((N, M)) * std


def normal_bf16(N: int, M: int, seed: int, std: float = 1.0) -> np.ndarray:
    """Entries i.i.d. N(0, std^2) rounded to bfloat16; uint16 bit patterns."""
    return f32_to_bf16_bits(_normal(np.random.default_rng(seed), (N, M), std))


def normal_f32(N: int, M: int, seed: int, std: float = 1.0, tf32_exact: bool = False) -> np.ndarray:
    """Entries i.i.d. N(0, std^2), binary32; with ``tf32_exact`` the low 13 bits are cleared."""
    v = _normal(np.random.default_rng(seed), (N, M), std)
    return f32_keep_tf32_bits(v) if tf32_exact else v


def small_int_f32(N: int, M: int, seed: int, lo: int = -2, hi: int = 2) -> np.ndarray:
    """Integer entries in [lo, hi] stored as binary32 (exact in TF32)."""
    return np.random.default_rng(seed).integers(lo, hi + 1, size=(N, M)).astype(np.float32)


def normal_e4m3(N: int, M: int, seed: int, std: float = 1.0) -> np.ndarray:
    """Entries i.i.d. N(0, std^2) rounded to FP8 E4M3; uint8 bytes."""
    return f32_to_e4m3_bits(_normal(np.random.default_rng(seed), (N, M), std))


def small_int_e4m3(N: int, M: int, seed: int, lo: int = -2, hi: int = 2) -> np.ndarray:
    """Integer entries in [lo, hi] as FP8 E4M3 bytes (exactly representable)."""
    return f32_to_e4m3_bits(np.random.default_rng(seed).integers(lo, hi + 1, size=(N, M)).astype(np.float32))


def normal_f16(N: int, M: int, seed: int, std: float = 1.0) -> np.ndarray:
    """Entries i.i.d. N(0, std^2) rounded to binary16; uint16 bit patterns."""
    return f32_to_f16_bits(_normal(np.random.default_rng(seed), (N, M), std))


def small_int_f16(N: int, M: int, seed: int, lo: int = -2, hi: int = 2) -> np.ndarray:
    """Integer entries in [lo, hi] as binary16 bit patterns (exactly representable)."""
    return f32_to_f16_bits(np.random.default_rng(seed).integers(lo, hi + 1, size=(N, M)).astype(np.float32))


def small_int_f64(N: int, M: int, seed: int, lo: int = -2, hi: int = 2) -> np.ndarray:
    """Integer entries in [lo, hi] stored as binary64 (every partial sum is exact)."""
    return np.random.default_rng(seed).integers(lo, hi + 1, size=(N, M)).astype(np.float64)


def normal_c128(N: int, M: int, seed: int, std: float = 1.0) -> np.ndarray:
    """Complex N x M with independent N(0, std^2) real and imaginary parts (complex128)."""
    rng = np.random.default_rng(seed)
    out = np.empty((N, M), dtype=np.complex128)
    out.real = rng.standard_normal((N, M)) * std
    out.imag = rng.standard_normal((N, M)) * std
    return out


def small_int_c128(N: int, M: int, seed: int, lo: int = -2, hi: int = 2) -> np.ndarray:
    """Gaussian integers with both parts in [lo, hi] (complex128): every sum of products is exact."""
    rng = np.random.default_rng(seed)
    out = np.empty((N, M), dtype=np.complex128)
    out.real = rng.integers(lo, hi + 1, size=(N, M))
    out.imag = rng.integers(lo, hi + 1, size=(N, M))
    return out


def random_c128(N: int, seed: int, ldc: Optional[int] = None) -> np.ndarray:
    """A complex N x ldc array for C (uniform parts in [-1, 1)); the caller reads its lower triangle."""
    rng = np.random.default_rng(seed)
    ldc = N if ldc is None else ldc
    out = np.empty((N, ldc), dtype=np.complex128)
    out.real = rng.uniform(-1.0, 1.0, size=(N, ldc))
    out.imag = rng.uniform(-1.0, 1.0, size=(N, ldc))
    return out


def small_int_bf16(N: int, M: int, seed: int, lo: int = -2, hi: int = 2) -> np.ndarray:
    """Integer entries in [lo, hi] as bfloat16 bit patterns (exactly representable)."""
    v = np.random.default_rng(seed).integers(lo, hi + 1, size=(N, M)).astype(np.float32)
    return f32_to_bf16_bits(v)


def ones(N: int, M: int, dtype: int) -> np.ndarray:
    """All-ones A in the storage type of ``dtype``."""
    if dtype == DTYPE_F64:
        return np.ones((N, M), dtype=np.float64)
    if dtype == DTYPE_TF32_F32:
        return np.ones((N, M), dtype=np.float32)
    if dtype == DTYPE_E4M3_F32:
        return f32_to_e4m3_bits(np.ones((N, M), dtype=np.float32))
    if dtype == DTYPE_F16_F32:
        return f32_to_f16_bits(np.ones((N, M), dtype=np.float32))
    return f32_to_bf16_bits(np.ones((N, M), dtype=np.float32))


def to_storage(values: np.ndarray, dtype: int) -> np.ndarray:
    """Values (exactly representable in the target type) -> storage array for A."""
    if dtype == DTYPE_F64:
        return np.ascontiguousarray(values, dtype=np.float64)
    if dtype == DTYPE_TF32_F32:
        return np.ascontiguousarray(values, dtype=np.float32)
    if dtype == DTYPE_E4M3_F32:
        return f32_to_e4m3_bits(np.asarray(values, dtype=np.float32))
    if dtype == DTYPE_F16_F32:
        return f32_to_f16_bits(np.asarray(values, dtype=np.float32))
    return f32_to_bf16_bits(np.asarray(values, dtype=np.float32))


def c_storage_dtype(dtype: int):
    return np.float64 if dtype == DTYPE_F64 else np.float32


def random_c(N: int, seed: int, dtype: int, ldc: Optional[int] = None) -> np.ndarray:
    """A full N x ldc prior value of C (both triangles filled; N(0,1))."""
    ldc = N if ldc is None else ldc
    c = np.random.default_rng(seed).standard_normal((N, ldc))
    return c.astype(c_storage_dtype(dtype))


@dataclass
class Workload:
    """One benchmark configuration: shapes, scalars, type and the recipe for A."""
    name: str
    N: int
    M: int
    dtype: int
    alpha: float
    beta: float
    seed: int
    dist: str            # "uniform", "normal"
    std: float = 1.0

    def make_A(self) -> np.ndarray:
        if self.dtype == DTYPE_F64:
            if self.dist == "uniform":
                return uniform_f64(self.N, self.M, self.seed)
            return normal_f64(self.N, self.M, self.seed, self.std)
        if self.dtype == DTYPE_TF32_F32:
            return normal_f32(self.N, self.M, self.seed, self.std)
        if self.dtype == DTYPE_E4M3_F32:
            return normal_e4m3(self.N, self.M, self.seed, self.std)
        if self.dtype == DTYPE_F16_F32:
            return normal_f16(self.N, self.M, self.seed, self.std)
        return normal_bf16(self.N, self.M, self.seed, self.std)

    @property
    def flops(self) -> int:
        return self.N * (self.N + 1) * self.M


# The four single-call configurations (the fifth is a sweep, see cholesky_sweep_*).
CONFIGS = {
    "c1": Workload("c1_f64_512x256", 512, 256, DTYPE_F64, 1.0, 0.0, 0, "uniform"),
    "c2": Workload("c2_f64_4096x4096", 4096, 4096, DTYPE_F64, 1.0, 0.0, 1, "normal"),
    "c3": Workload("c3_bf16_16384x4096", 16384, 4096, DTYPE_BF16_F32, 1.0, 0.0, 2, "normal"),
    "c4": Workload("c4_bf16_2048x262144", 2048, 262144, DTYPE_BF16_F32, 1.0, 0.0, 3, "normal",
                   std=2.0 ** -9),
}

# Cholesky-shaped trailing-update sweep: n = n_max, n_max - step, ..., step; inner
# dimension 512; alpha = -1, beta = 1; seed 4.
SWEEP_K = 512
SWEEP_SEED = 4


def sweep_sizes(n_max: int = 32768, step: int = 512):
    return list(range(n_max, 0, -step))


def sweep_panel(n: int, n_max: int = 32768) -> np.ndarray:
    """A_n: n x 512 binary64, N(0,1)/sqrt(512); one independent stream per n."""
    rng = np.random.default_rng([SWEEP_SEED, 1, n, n_max])
    return rng.standard_normal((n, SWEEP_K)) / np.sqrt(float(SWEEP_K))


def sweep_factor(n_max: int = 32768) -> np.ndarray:
    """G: n_max x 512 binary64 N(0,1).  The swept matrix is n_max*I + G G^T / 512;
    forming that product is input preparation and is left to the caller."""
    rng = np.random.default_rng([SWEEP_SEED, 0, n_max])
    return rng.standard_normal((n_max, SWEEP_K))
