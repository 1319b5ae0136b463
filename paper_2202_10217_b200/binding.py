"""Thin ctypes binding of libtbsyrk.so: same names as the C ABI, argument
marshalling only.  Every step of the computation runs in the library's CUDA
kernels; there is no CPU or PyTorch fallback, and loading fails loudly when the
shared library has not been built.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libtbsyrk.so")

DTYPE_F64 = 0
DTYPE_BF16_F32 = 1
DTYPE_TF32_F32 = 2
DTYPE_E4M3_F32 = 3
DTYPE_F16_F32 = 4
UPLO_LOWER, UPLO_UPPER = 0, 1
OP_N, OP_T = 0, 1
SCHEDULE_TBS = 0
SCHEDULE_SQUARE = 1
SCHEDULE_PAIR_SQUARE = 2
SCHEDULE_AUTO = 3
SCHEDULE_DEFAULT = SCHEDULE_AUTO      # what the library starts with
SCHEDULE_NAME = {SCHEDULE_TBS: "tbs", SCHEDULE_SQUARE: "square", SCHEDULE_PAIR_SQUARE: "pair_square"}
ITEM_TRI, ITEM_RECT, ITEM_DIAG = 0, 1, 2
MAX_SEG, MAX_TILE = 8, 16

EXPORTS = [
    "syrk_lower", "syrk_lower_tn", "syrk_ex", "syr2k_lower", "syr2k_lower_ex", "herk_lower", "syrk_lower_batched", "syrk_lower_host", "syrk_plan_prepare", "syrk_plan_prepare_stream", "syrk_effective_schedule",
    "syrk_lower_bf16_static_status", "syrk_set_host_pipeline", "syrk_host_pipeline_for", "syrk_pack_lower", "syrk_unpack_lower_axpby", "syrk_shutdown", "syrk_last_status",
    "syrk_strerror", "syrk_set_schedule", "syrk_set_split_k", "syrk_set_f64_tail_split", "syrk_set_f64_launch", "syrk_get_schedule_stats",
    "syrk_probe_f64_mma_peak", "syrk_selftest_bounded_wait", "syrk_lower_bf16_static", "cholesky_lower", "cholesky_last_info",
    "tbs_plan_build", "tbs_plan_balance", "tbs_plan_num_items", "tbs_plan_item", "tbs_plan_free", "tbs_plan_simulate",
]


class ScheduleStats(ctypes.Structure):
    _fields_ = [("tile", ctypes.c_int32), ("k", ctypes.c_int32), ("c", ctypes.c_int32),
                ("split_k", ctypes.c_int32), ("n_tiles", ctypes.c_int64), ("items", ctypes.c_int64),
                ("tri_items", ctypes.c_int64), ("rect_items", ctypes.c_int64),
                ("diag_items", ctypes.c_int64), ("tri_tiles", ctypes.c_int64),
                ("all_tiles", ctypes.c_int64), ("a_loads", ctypes.c_int64),
                ("c_elems", ctypes.c_int64), ("s_acc", ctypes.c_int64), ("s_total", ctypes.c_int64),
                ("effective_schedule", ctypes.c_int32), ("launches", ctypes.c_int32)]

    def as_dict(self):
        return {name: int(getattr(self, name)) for name, _ in self._fields_}


class SyrkError(RuntimeError):
    def __init__(self, code: int):
        self.code = code
        super().__init__("tbsyrk error %d: %s" % (code, strerror(code)))


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded shared library (raises if it is not built)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError("libtbsyrk.so is missing: run `python -m paper_2202_10217_b200.build` "
                              "(there is no fallback implementation)")
        L = ctypes.CDLL(LIB_PATH)
        i64, i32, dbl, vp, ci = ctypes.c_int64, ctypes.c_int32, ctypes.c_double, ctypes.c_void_p, ctypes.c_int
        L.syrk_lower.restype = ci
        L.syrk_lower.argtypes = [i64, i64, vp, i64, vp, i64, dbl, dbl, ci, vp]
        L.syrk_lower_tn.restype = ci
        L.syrk_lower_tn.argtypes = [i64, i64, vp, i64, vp, i64, dbl, dbl, ci, vp]
        L.syrk_ex.restype = ci
        L.syrk_ex.argtypes = [ci, ci, i64, i64, vp, i64, vp, i64, dbl, dbl, ci, vp]
        L.herk_lower.restype = ci
        L.herk_lower.argtypes = [i64, i64, vp, i64, vp, i64, dbl, dbl, vp]
        L.syr2k_lower.restype = ci
        L.syr2k_lower.argtypes = [i64, i64, vp, i64, vp, i64, vp, i64, dbl, dbl, vp]
        L.syr2k_lower_ex.restype = ci
        L.syr2k_lower_ex.argtypes = [i64, i64, vp, i64, vp, i64, vp, i64, dbl, dbl, ci, vp]
        L.syrk_lower_batched.restype = ci
        L.syrk_lower_batched.argtypes = [i64, i64, i64, vp, i64, i64, vp, i64, i64, dbl, dbl, ci, vp]
        L.syrk_lower_host.restype = ci
        L.syrk_lower_host.argtypes = [i64, i64, vp, i64, vp, i64, dbl, dbl, ci]
        L.syrk_plan_prepare.restype = ci
        L.syrk_plan_prepare.argtypes = [i64, i64, ci]
        L.syrk_plan_prepare_stream.restype = ci
        L.syrk_plan_prepare_stream.argtypes = [i64, i64, ci, vp]
        L.syrk_effective_schedule.restype = ci
        L.syrk_effective_schedule.argtypes = [i64, i64, ci]
        L.syrk_lower_bf16_static_status.restype = ci
        L.syrk_lower_bf16_static_status.argtypes = []
        L.syrk_set_host_pipeline.restype = ci
        L.syrk_set_host_pipeline.argtypes = [ci]
        L.syrk_host_pipeline_for.restype = ci
        L.syrk_host_pipeline_for.argtypes = [i64, i64, ci]
        L.syrk_pack_lower.restype = ci
        L.syrk_pack_lower.argtypes = [i64, vp, i64, ci, vp, vp]
        L.syrk_unpack_lower_axpby.restype = ci
        L.syrk_unpack_lower_axpby.argtypes = [i64, i64, i64, vp, dbl, vp, i64, ci, vp]
        L.syrk_shutdown.restype = None
        L.syrk_shutdown.argtypes = []
        L.syrk_last_status.restype = ci
        L.syrk_last_status.argtypes = [vp]
        L.syrk_strerror.restype = ctypes.c_char_p
        L.syrk_strerror.argtypes = [ci]
        L.syrk_set_schedule.restype = ci
        L.syrk_set_schedule.argtypes = [ci]
        L.syrk_set_split_k.restype = ci
        L.syrk_set_split_k.argtypes = [ci]
        L.syrk_set_f64_tail_split.restype = ci
        L.syrk_set_f64_tail_split.argtypes = [ci, i64]
        L.syrk_set_f64_launch.restype = ci
        L.syrk_set_f64_launch.argtypes = [ci]
        L.syrk_get_schedule_stats.restype = ci
        L.syrk_get_schedule_stats.argtypes = [i64, i64, ci, ctypes.POINTER(ScheduleStats)]
        L.syrk_probe_f64_mma_peak.restype = ci
        L.syrk_probe_f64_mma_peak.argtypes = [ci, ctypes.POINTER(dbl)]
        L.syrk_selftest_bounded_wait.restype = ci
        L.syrk_selftest_bounded_wait.argtypes = [vp]
        L.syrk_lower_bf16_static.restype = ci
        L.syrk_lower_bf16_static.argtypes = [i64, i64, vp, i64, vp, i64, dbl, dbl, ci, vp]
        L.cholesky_lower.restype = ci
        L.cholesky_lower.argtypes = [i64, vp, i64, i64, vp]
        L.cholesky_last_info.restype = i64
        L.cholesky_last_info.argtypes = [vp]
        L.tbs_plan_build.restype = vp
        L.tbs_plan_build.argtypes = [i64, ci, ci, ci, ci, ci]
        L.tbs_plan_balance.restype = ci
        L.tbs_plan_balance.argtypes = [vp, ci]
        L.tbs_plan_num_items.restype = i64
        L.tbs_plan_num_items.argtypes = [vp]
        L.tbs_plan_item.restype = ci
        L.tbs_plan_item.argtypes = [vp, i64, ctypes.POINTER(i32), ctypes.POINTER(i32),
                                    ctypes.POINTER(i32), ctypes.POINTER(i32), ctypes.POINTER(i32),
                                    ctypes.POINTER(i32)]
        L.tbs_plan_free.restype = None
        L.tbs_plan_free.argtypes = [vp]
        L.tbs_plan_simulate.restype = ci
        L.tbs_plan_simulate.argtypes = [vp, i64, i64, ci, ctypes.POINTER(i64), ctypes.POINTER(i64),
                                        ctypes.POINTER(i32), ctypes.POINTER(i32), ctypes.POINTER(i32)]
        _lib = L
    return _lib


def strerror(code: int) -> str:
    return lib().syrk_strerror(int(code)).decode()


def _check(code: int) -> None:
    if code != 0:
        raise SyrkError(code)


def _ptr(x) -> Optional[int]:
    """Raw address of a torch tensor / numpy array / int / None."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        return int(x.data_ptr())
    if hasattr(x, "ctypes"):
        return int(x.ctypes.data)
    raise TypeError("cannot take the address of %r" % type(x))


def syrk_lower(N: int, M: int, A, lda: int, C, ldc: int, alpha: float, beta: float, dtype: int,
               stream: Optional[int] = None) -> None:
    """Enqueue C_lower <- alpha * A A^T + beta * C_lower on `stream` (device pointers).

    `A` and `C` are torch CUDA tensors (or raw device addresses); `stream` is a raw
    cudaStream_t, by default torch's current stream.
    """
    if stream is None:
        import torch
        stream = torch.cuda.current_stream().cuda_stream
    _check(lib().syrk_lower(N, M, _ptr(A), lda, _ptr(C), ldc, float(alpha), float(beta), dtype, stream))


def syrk_lower_tn(N: int, M: int, A, lda: int, C, ldc: int, alpha: float, beta: float, dtype: int,
                  stream: Optional[int] = None) -> None:
    """Enqueue C_lower <- alpha * A^T A + beta * C_lower, A an M x N row-major device array."""
    if stream is None:
        import torch
        stream = torch.cuda.current_stream().cuda_stream
    _check(lib().syrk_lower_tn(N, M, _ptr(A), lda, _ptr(C), ldc, float(alpha), float(beta), dtype, stream))


def syrk_ex(uplo: int, trans: int, N: int, M: int, A, lda: int, C, ldc: int, alpha: float, beta: float,
            dtype: int, stream: Optional[int] = None) -> None:
    """General form: stored triangle `uplo` of C <- alpha * op(A) op(A)^T + beta * C (device pointers)."""
    if stream is None:
        import torch
        stream = torch.cuda.current_stream().cuda_stream
    _check(lib().syrk_ex(uplo, trans, N, M, _ptr(A), lda, _ptr(C), ldc, float(alpha), float(beta), dtype, stream))


def syr2k_lower(N: int, M: int, A, lda: int, Bm, ldb: int, C, ldc: int, alpha: float, beta: float,
                stream: Optional[int] = None) -> None:
    """Enqueue C_lower <- alpha * (A B^T + B A^T) + beta * C_lower (binary64, device pointers)."""
    if stream is None:
        import torch
        stream = torch.cuda.current_stream().cuda_stream
    _check(lib().syr2k_lower(N, M, _ptr(A), lda, _ptr(Bm), ldb, _ptr(C), ldc, float(alpha), float(beta), stream))


def herk_lower(N: int, M: int, A, lda: int, C, ldc: int, alpha: float, beta: float,
               stream: Optional[int] = None) -> None:
    """Enqueue C_lower <- alpha * A A^H + beta * C_lower (complex128 as (re, im) pairs, device pointers,
    pitches in complex entries)."""
    if stream is None:
        import torch
        stream = torch.cuda.current_stream().cuda_stream
    _check(lib().herk_lower(N, M, _ptr(A), lda, _ptr(C), ldc, float(alpha), float(beta), stream))


def syr2k_lower_ex(N: int, M: int, A, lda: int, Bm, ldb: int, C, ldc: int, alpha: float, beta: float, dtype: int,
                   stream: Optional[int] = None) -> None:
    """Enqueue C_lower <- alpha * (A B^T + B A^T) + beta * C_lower for any dtype of the library (device pointers)."""
    if stream is None:
        import torch
        stream = torch.cuda.current_stream().cuda_stream
    _check(lib().syr2k_lower_ex(N, M, _ptr(A), lda, _ptr(Bm), ldb, _ptr(C), ldc, float(alpha), float(beta), dtype, stream))


def syrk_lower_batched(batch: int, N: int, M: int, A, lda: int, stride_a: int, C, ldc: int, stride_c: int,
                       alpha: float, beta: float, dtype: int, stream: Optional[int] = None) -> None:
    """`batch` independent updates C_b = alpha * A_b A_b^T + beta * C_b on device memory; strides in elements."""
    if stream is None:
        import torch
        stream = torch.cuda.current_stream().cuda_stream
    _check(lib().syrk_lower_batched(batch, N, M, _ptr(A), lda, stride_a, _ptr(C), ldc, stride_c, float(alpha),
                                    float(beta), dtype, stream))


def syrk_lower_host(N: int, M: int, A, lda: int, C, ldc: int, alpha: float, beta: float,
                    dtype: int) -> None:
    """Same operation on HOST buffers (numpy arrays, CPU tensors or raw addresses);
    copies in, computes on the GPU, copies the lower triangle back, and waits."""
    _check(lib().syrk_lower_host(N, M, _ptr(A), lda, _ptr(C), ldc, float(alpha), float(beta), dtype))


def syrk_lower_bf16_static(N: int, M: int, A, lda: int, C, ldc: int, alpha: float, beta: float,
                           slices: int, stream: Optional[int] = None) -> None:
    """K-split BF16 update that allocates nothing: its work list and partial tiles live in
    fixed device arrays of the library (for callers that cannot let a library call
    cudaMalloc).  Raises SyrkError(-10) when the problem exceeds those arrays.  Calls share
    the arrays, so overlapping calls must be serialised by the caller."""
    if stream is None:
        import torch
        stream = torch.cuda.current_stream().cuda_stream
    _check(lib().syrk_lower_bf16_static(N, M, _ptr(A), lda, _ptr(C), ldc, float(alpha), float(beta),
                                        int(slices), stream))


def cholesky_lower(N: int, A, lda: int, block: int = 0, stream: Optional[int] = None) -> None:
    """Enqueue the in-place lower Cholesky factorisation (Large Block Cholesky) of the FP64 device
    matrix A; check cholesky_last_info() after synchronising."""
    if stream is None:
        import torch
        stream = torch.cuda.current_stream().cuda_stream
    _check(lib().cholesky_lower(N, _ptr(A), lda, block, stream))


def cholesky_last_info(stream: Optional[int] = None) -> int:
    """0, or k + 1 for the first non-positive pivot k of the last factorisation (after a sync)."""
    return int(lib().cholesky_last_info(stream))


def syrk_plan_prepare(N: int, M: int, dtype: int) -> None:
    _check(lib().syrk_plan_prepare(N, M, dtype))


def syrk_plan_prepare_stream(N: int, M: int, dtype: int, stream: Optional[int] = None) -> None:
    """Create ahead of time what syrk_lower(N, M, ..., dtype) on `stream` (default: torch's current
    stream) would allocate."""
    if stream is None:
        import torch
        stream = torch.cuda.current_stream().cuda_stream
    _check(lib().syrk_plan_prepare_stream(N, M, dtype, stream))


def syrk_effective_schedule(N: int, M: int, dtype: int) -> int:
    """SCHEDULE_TBS, SCHEDULE_SQUARE or SCHEDULE_PAIR_SQUARE: what a call with these sizes runs (host only)."""
    r = int(lib().syrk_effective_schedule(N, M, dtype))
    if r < 0:
        raise SyrkError(r)
    return r


HOST_AUTO, HOST_ROW_BANDS, HOST_COLUMN_BLOCKS = 0, 1, 2


def syrk_set_host_pipeline(mode: int) -> None:
    _check(lib().syrk_set_host_pipeline(mode))


def syrk_host_pipeline_for(N: int, M: int, c_is_page_locked: bool) -> int:
    """HOST_ROW_BANDS (square-block list) or HOST_COLUMN_BLOCKS (the schedule of syrk_lower): what
    syrk_lower_host does with these sizes (host only)."""
    r = int(lib().syrk_host_pipeline_for(N, M, 1 if c_is_page_locked else 0))
    if r < 0:
        raise SyrkError(r)
    return r


def syrk_pack_lower(N: int, C, ldc: int, dtype: int, packed, stream: Optional[int] = None) -> None:
    """packed[i (i + 1) / 2 + j] <- C[i][j], j <= i (device pointers; enqueues)."""
    if stream is None:
        import torch
        stream = torch.cuda.current_stream().cuda_stream
    _check(lib().syrk_pack_lower(N, _ptr(C), ldc, dtype, _ptr(packed), stream))


def syrk_unpack_lower_axpby(N: int, first: int, count: int, packed, beta: float, C, ldc: int, dtype: int,
                            stream: Optional[int] = None) -> None:
    """C[i][j] <- packed value + beta * C[i][j] for the packed entries first .. first + count - 1."""
    if stream is None:
        import torch
        stream = torch.cuda.current_stream().cuda_stream
    _check(lib().syrk_unpack_lower_axpby(N, first, count, _ptr(packed), float(beta), _ptr(C), ldc, dtype, stream))


def syrk_lower_bf16_static_status() -> int:
    """0, or -8 once after a bounded wait ran out inside syrk_lower_bf16_static (after a sync)."""
    return int(lib().syrk_lower_bf16_static_status())


def syrk_shutdown() -> None:
    lib().syrk_shutdown()


def syrk_last_status(stream: Optional[int] = None) -> int:
    return int(lib().syrk_last_status(stream))


def syrk_selftest_bounded_wait(stream: Optional[int] = None) -> None:
    """Enqueue the kernel whose bounded wait runs out on purpose (about two seconds)."""
    if stream is None:
        import torch
        stream = torch.cuda.current_stream().cuda_stream
    _check(lib().syrk_selftest_bounded_wait(stream))


def syrk_set_schedule(schedule: int) -> None:
    _check(lib().syrk_set_schedule(schedule))


F64_LAUNCH_AUTO, F64_LAUNCH_PER_ITEM, F64_LAUNCH_PERSISTENT = 0, 1, 2


def syrk_set_f64_launch(mode: int) -> None:
    _check(lib().syrk_set_f64_launch(mode))


def syrk_set_f64_tail_split(slices: int, tail_items: int = 0) -> None:
    """0: automatic; 1: never; >= 2: the last `tail_items` items of an FP64 list run in that many K-slices."""
    _check(lib().syrk_set_f64_tail_split(slices, tail_items))


def syrk_set_split_k(slices: int) -> None:
    _check(lib().syrk_set_split_k(slices))


def syrk_get_schedule_stats(N: int, M: int, dtype: int) -> dict:
    st = ScheduleStats()
    _check(lib().syrk_get_schedule_stats(N, M, dtype, ctypes.byref(st)))
    return st.as_dict()


def syrk_probe_f64_mma_peak(iters: int = 20000) -> float:
    """Measured FP64 tensor-core throughput of the current GPU, TFLOP/s."""
    out = ctypes.c_double()
    _check(lib().syrk_probe_f64_mma_peak(iters, ctypes.byref(out)))
    return float(out.value)


class Plan:
    """Host-side work list (tbs_plan_* calls); no device needed."""

    def __init__(self, n_tiles: int, k: int, rect_rows: int, rect_cols: int, diag_side: int,
                 schedule: int = SCHEDULE_TBS):
        self._h = lib().tbs_plan_build(n_tiles, k, rect_rows, rect_cols, diag_side, schedule)
        if not self._h:
            raise SyrkError(-7)
        self.n_tiles = n_tiles

    def balance(self, slots: int) -> None:
        _check(lib().tbs_plan_balance(self._h, slots))

    def __len__(self) -> int:
        return int(lib().tbs_plan_num_items(self._h))

    def item(self, index: int):
        """(kind, [segments], [(x_slot, y_slot), ...])"""
        i32 = ctypes.c_int32
        kind, n_seg, n_tile = i32(), i32(), i32()
        seg = (i32 * MAX_SEG)()
        tx = (i32 * MAX_TILE)()
        ty = (i32 * MAX_TILE)()
        _check(lib().tbs_plan_item(self._h, index, ctypes.byref(kind), ctypes.byref(n_seg), seg,
                                   ctypes.byref(n_tile), tx, ty))
        return (kind.value, list(seg[:n_seg.value]),
                [(tx[t], ty[t]) for t in range(n_tile.value)])

    def simulate(self, N: int, M: int, b: int) -> dict:
        i64, i32 = ctypes.c_int64, ctypes.c_int32
        a, c = i64(), i64()
        lo, hi, up = i32(), i32(), i32()
        _check(lib().tbs_plan_simulate(self._h, N, M, b, ctypes.byref(a), ctypes.byref(c),
                                       ctypes.byref(lo), ctypes.byref(hi), ctypes.byref(up)))
        return {"a_loads": a.value, "c_loads": c.value, "min_cover": lo.value,
                "max_cover": hi.value, "upper_cover": up.value}

    def close(self) -> None:
        if self._h:
            lib().tbs_plan_free(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
