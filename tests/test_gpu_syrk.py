"""GPU parity: the CUDA path, called through the C ABI, against the CPU reference,
entry by entry on the same seeded inputs.

Tolerance (binary64 reference of the exact products):
    |C_gpu - C_ref| <= tol * M * (|alpha| * (|A||A|^T)_ij + |beta| * |C_in,ij|)
with tol = 8 * 2^-53 (FP64) and 4 * 2^-24 (BF16 inputs, FP32 accumulation).
Integer-valued inputs must match bit for bit whatever the summation order.
"""
import numpy as np
import pytest
import torch

from oracle import syrk as O
from paper_2202_10217_b200 import binding as B
from paper_2202_10217_b200 import inputs as I

from gpu_util import assert_within_tolerance, run_case

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def triangle_block_schedule():
    """This file is the parity suite of the triangle-block kernels: the sizes an entry-by-entry reference
    can check are all below the size at which the default schedule starts to use them for the tcgen05
    types, so the schedule is pinned here (the default is covered by test_gpu_default_schedule.py,
    test_gpu_configs.py and the random sweep)."""
    B.syrk_set_schedule(B.SCHEDULE_TBS)
    yield
    B.syrk_set_schedule(B.SCHEDULE_DEFAULT)


BOTH = [B.DTYPE_F64, B.DTYPE_BF16_F32, B.DTYPE_TF32_F32, B.DTYPE_E4M3_F32,
        B.DTYPE_F16_F32]                                                     # every input type of the library
DT = pytest.mark.parametrize("dtype", BOTH, ids=["f64", "bf16", "tf32", "e4m3", "f16"])
A_NUMPY = {B.DTYPE_F64: np.float64, B.DTYPE_BF16_F32: np.uint16, B.DTYPE_TF32_F32: np.float32,
           B.DTYPE_E4M3_F32: np.uint8, B.DTYPE_F16_F32: np.uint16}
ALIGN_ELEMS = {B.DTYPE_F64: 2, B.DTYPE_BF16_F32: 8, B.DTYPE_TF32_F32: 4, B.DTYPE_E4M3_F32: 16,
               B.DTYPE_F16_F32: 8}                                           # elements per 16 bytes


def make_A(N, M, dtype, seed, kind="normal"):
    """Real-valued TF32 inputs keep their low-order bits: the library must ignore them."""
    if kind == "int":
        return {B.DTYPE_F64: I.small_int_f64, B.DTYPE_BF16_F32: I.small_int_bf16,
                B.DTYPE_TF32_F32: I.small_int_f32, B.DTYPE_E4M3_F32: I.small_int_e4m3,
                B.DTYPE_F16_F32: I.small_int_f16}[dtype](N, M, seed)
    return {B.DTYPE_F64: I.normal_f64, B.DTYPE_BF16_F32: I.normal_bf16, B.DTYPE_TF32_F32: I.normal_f32,
            B.DTYPE_E4M3_F32: I.normal_e4m3, B.DTYPE_F16_F32: I.normal_f16}[dtype](N, M, seed)


# Sizes: below one tile, exact tiles, ragged tails in N and M, several tiles, and sizes
# large enough for triangle blocks (FP64: >= 30 tile rows of 32; BF16: >= 6 tile rows of 128).
SIZES_F64 = [(1, 1), (5, 3), (31, 17), (32, 16), (33, 50), (100, 64), (257, 130), (512, 256),
             (1000, 70), (1300, 40)]
SIZES_BF16 = [(1, 8), (5, 24), (127, 64), (128, 64), (129, 72), (300, 200), (512, 256),
              (777, 136), (1100, 320), (2050, 72)]
SIZES_TF32 = [(1, 4), (5, 12), (127, 32), (128, 64), (129, 36), (300, 100), (512, 256),
              (777, 68), (1100, 160), (2050, 44)]
SIZES_E4M3 = [(1, 16), (5, 48), (127, 128), (128, 256), (129, 144), (300, 400), (512, 512),
              (777, 272), (1100, 640), (2050, 144), (300, 77)]


def sizes(dtype):
    return {B.DTYPE_F64: SIZES_F64, B.DTYPE_BF16_F32: SIZES_BF16, B.DTYPE_TF32_F32: SIZES_TF32,
            B.DTYPE_E4M3_F32: SIZES_E4M3, B.DTYPE_F16_F32: SIZES_BF16}[dtype]


@DT
def test_real_inputs_within_tolerance(dtype):
    for n, (N, M) in enumerate(sizes(dtype)):
        A = make_A(N, M, dtype, seed=100 + n)
        got, ref, bound = run_case(A, dtype, 1.0, 0.0)
        assert_within_tolerance(got, ref, bound, M, 1.0, 0.0, None, dtype)


@DT
def test_integer_inputs_are_bit_exact(dtype):
    for n, (N, M) in enumerate(sizes(dtype)):
        A = make_A(N, M, dtype, seed=200 + n, kind="int")
        got, ref, bound = run_case(A, dtype, 1.0, 0.0)
        assert_within_tolerance(got, ref, bound, M, 1.0, 0.0, None, dtype, exact=True)


@DT
@pytest.mark.parametrize("alpha,beta", [(-1.0, 1.0), (0.0, 1.0), (0.0, 0.0), (2.5, -0.5), (1.0, 2.0),
                                        (0.0, -3.0)])
def test_alpha_beta(dtype, alpha, beta):
    N, M = (1000, 48) if dtype == B.DTYPE_F64 else (900, 128)
    A = make_A(N, M, dtype, seed=7, kind="int")
    Cin = (np.random.default_rng(9).integers(-8, 9, size=(N, N)) * 2).astype(I.c_storage_dtype(dtype))
    got, ref, bound = run_case(A, dtype, alpha, beta, Cin=Cin)
    if beta == 0.0:
        ref, bound = O.syrk_lower(A, None, alpha, 0.0, dtype)
    assert_within_tolerance(got, ref, bound, M, alpha, beta, Cin, dtype, exact=True)
    A = make_A(N, M, dtype, seed=8)
    Cin = I.random_c(N, 10, dtype)
    got, ref, bound = run_case(A, dtype, alpha, beta, Cin=Cin)
    assert_within_tolerance(got, ref, bound, M, alpha, beta, Cin, dtype)


@DT
def test_beta_zero_ignores_nan_in_C(dtype):
    N, M = (200, 40) if dtype == B.DTYPE_F64 else (300, 64)
    A = make_A(N, M, dtype, seed=3)
    got, ref, bound = run_case(A, dtype, 1.0, 0.0, poison=True)
    assert_within_tolerance(got, ref, bound, M, 1.0, 0.0, None, dtype)


@DT
def test_pitches_and_offsets(dtype):
    N, M = (300, 50) if dtype == B.DTYPE_F64 else (400, 100)
    A = make_A(N, M, dtype, seed=4)
    Cin = I.random_c(N, 5, dtype)
    step = ALIGN_ELEMS[dtype]                         # keeps A 16-byte aligned (TMA path)
    got, ref, bound = run_case(A, dtype, -1.0, 1.0, Cin=Cin, lda=M - M % step + 4 * step, ldc=N + 37,
                               a_offset=3 * step, c_offset=5)
    assert_within_tolerance(got, ref, bound, M, -1.0, 1.0, Cin, dtype)


@DT
def test_unaligned_A_takes_the_plain_kernel(dtype):
    N, M = (150, 33) if dtype == B.DTYPE_F64 else (150, 77)
    A = make_A(N, M, dtype, seed=6)
    Cin = I.random_c(N, 5, dtype)
    got, ref, bound = run_case(A, dtype, 1.5, 0.5, Cin=Cin, lda=M + 3,
                               a_offset=1)
    assert_within_tolerance(got, ref, bound, M, 1.5, 0.5, Cin, dtype)


@DT
def test_closed_forms(dtype):
    N, M = (700, 96) if dtype == B.DTYPE_F64 else (640, 256)
    got, ref, bound = run_case(I.ones(N, M, dtype), dtype, 1.0, 0.0)
    assert np.all(got[np.tril_indices(N)] == float(M))
    H = np.array([[1.0]])
    while H.shape[0] < 256:
        H = np.block([[H, H], [H, -H]])
    got, ref, bound = run_case(I.to_storage(H / 16.0, dtype), dtype, 1.0, 0.0)   # orthonormal rows
    assert np.array_equal(got[np.tril_indices(256)], np.eye(256)[np.tril_indices(256)])


@DT
def test_degenerate_sizes(dtype):
    cdt = I.c_storage_dtype(dtype)
    # M == 0: lower triangle <- beta * C
    A = np.zeros((40, 0), dtype=A_NUMPY[dtype])
    Cin = I.random_c(40, 1, dtype)
    got, _, _ = run_case(A, dtype, 1.0, 2.0, Cin=Cin)
    il = np.tril_indices(40)
    assert np.array_equal(got[il], (cdt(2.0) * Cin[il]).astype(np.float64))
    got, _, _ = run_case(A, dtype, 1.0, 0.0, poison=True)
    assert np.all(got[il] == 0.0)
    # N == 0 is a no-op
    B.syrk_lower(0, 16, None, 16, None, 1, 1.0, 0.0, dtype)


@DT
def test_square_schedule_gives_the_same_result(dtype):
    N, M = (1100, 64) if dtype == B.DTYPE_F64 else (1300, 192)
    A = make_A(N, M, dtype, seed=12, kind="int")
    try:
        B.syrk_set_schedule(B.SCHEDULE_SQUARE)
        got, ref, bound = run_case(A, dtype, 1.0, 0.0)
    finally:
        B.syrk_set_schedule(B.SCHEDULE_TBS)              # what the fixture of this file expects to undo
    assert_within_tolerance(got, ref, bound, M, 1.0, 0.0, None, dtype, exact=True)


@DT
def test_host_buffer_entry_point(dtype):
    N, M = (333, 45) if dtype == B.DTYPE_F64 else (500, 90)
    A = make_A(N, M, dtype, seed=13)
    Cin = I.random_c(N, 14, dtype)
    C = Cin.copy()
    B.syrk_lower_host(N, M, A, M, C, N, -1.0, 1.0, dtype)
    ref, bound = O.syrk_lower(A, Cin, -1.0, 1.0, dtype)
    assert_within_tolerance(C.astype(np.float64), ref, bound, M, -1.0, 1.0, Cin, dtype)
    iu = np.triu_indices(N, 1)
    assert np.array_equal(C[iu], Cin[iu])               # host upper triangle untouched


def test_shutdown_releases_everything_and_the_library_can_be_used_again():
    N, M = 300, 64
    A = make_A(N, M, B.DTYPE_F64, seed=21, kind="int")
    got1, ref, bound = run_case(A, B.DTYPE_F64, 1.0, 0.0)
    B.syrk_shutdown()
    B.syrk_plan_prepare(N, M, B.DTYPE_F64)               # rebuilds the cached work list
    got2, _, _ = run_case(A, B.DTYPE_F64, 1.0, 0.0)
    assert_within_tolerance(got2, ref, bound, M, 1.0, 0.0, None, B.DTYPE_F64, exact=True)
    assert np.array_equal(got1[np.tril_indices(N)], got2[np.tril_indices(N)])
    A16 = make_A(400, 128, B.DTYPE_BF16_F32, seed=22, kind="int")
    got, ref, bound = run_case(A16, B.DTYPE_BF16_F32, 1.0, 0.0)
    assert_within_tolerance(got, ref, bound, 128, 1.0, 0.0, None, B.DTYPE_BF16_F32, exact=True)


def test_two_streams_back_to_back():
    """Calls on two streams that do not overlap in C run correctly one after the other."""
    import torch
    N, M = 600, 96
    A = make_A(N, M, B.DTYPE_F64, seed=23, kind="int")
    dA = torch.from_numpy(A).cuda()
    outs = []
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    torch.cuda.synchronize()
    for s in streams:
        dC = torch.zeros((N, N), dtype=torch.float64, device="cuda")
        with torch.cuda.stream(s):
            B.syrk_lower(N, M, dA, M, dC, N, 1.0, 0.0, B.DTYPE_F64, stream=s.cuda_stream)
        outs.append(dC)
    torch.cuda.synchronize()
    assert B.syrk_last_status() == 0
    ref, _ = O.syrk_lower(A, None, 1.0, 0.0, B.DTYPE_F64)
    il = np.tril_indices(N)
    for dC in outs:
        assert np.array_equal(dC.cpu().numpy()[il], ref[il])


# ---- FP64 launch forms: one block per item / persistent blocks drawing items from a counter ----

@pytest.mark.parametrize("alpha,beta", [(1.0, 0.0), (-1.0, 1.0), (2.5, -0.5)])
def test_f64_launch_forms_agree_bit_for_bit(alpha, beta):
    """Both forms run every tile with the same arithmetic in the same order: identical bits,
    and both within tolerance of the reference.  Sizes span one item, a ragged edge, and a list
    several times longer than the SM count.  The persistent form writes C from separate warps: stores for
    beta = 0, one memory-side addition per entry for beta = 1 (the correctly rounded sum, as the other form's
    multiply-add gives), a multiply-add for any other beta."""
    for n, (N, M) in enumerate([(33, 50), (1000, 70), (1300, 40), (2500, 33), (5000, 48)]):
        A = make_A(N, M, B.DTYPE_F64, seed=300 + n)
        Cin = I.random_c(N, 7, B.DTYPE_F64) if beta != 0.0 else None
        outs = []
        for mode in (B.F64_LAUNCH_PER_ITEM, B.F64_LAUNCH_PERSISTENT, B.F64_LAUNCH_AUTO):
            try:
                B.syrk_set_f64_launch(mode)
                got, ref, bound = run_case(A, B.DTYPE_F64, alpha, beta, Cin)
            finally:
                B.syrk_set_f64_launch(B.F64_LAUNCH_AUTO)
            assert_within_tolerance(got, ref, bound, M, alpha, beta, Cin, B.DTYPE_F64)
            outs.append(got)
        il = np.tril_indices(N)
        assert np.array_equal(outs[0][il], outs[1][il]) and np.array_equal(outs[0][il], outs[2][il])


@pytest.mark.parametrize("alpha,beta", [(1.0, 0.0), (-1.0, 1.0), (0.5, 3.0)])
@pytest.mark.parametrize("ldc_pad,c_offset", [(3, 0), (0, 1), (5, 1)])
def test_f64_persistent_write_out_with_odd_pitch_or_offset_of_c(alpha, beta, ldc_pad, c_offset):
    """C off the 16-byte boundary or with an odd pitch: the write-out warps fall back to 8-byte accesses; same
    bits as the one-block-per-item form, canaries around C untouched (run_case checks them)."""
    N, M = 1400, 72
    A = make_A(N, M, B.DTYPE_F64, seed=340)
    Cin = I.random_c(N, 341, B.DTYPE_F64) if beta != 0.0 else None
    outs = []
    for mode in (B.F64_LAUNCH_PER_ITEM, B.F64_LAUNCH_PERSISTENT):
        try:
            B.syrk_set_f64_launch(mode)
            got, ref, bound = run_case(A, B.DTYPE_F64, alpha, beta, Cin, ldc=N + ldc_pad, c_offset=c_offset,
                                       poison=(beta == 0.0))
        finally:
            B.syrk_set_f64_launch(B.F64_LAUNCH_AUTO)
        assert_within_tolerance(got, ref, bound, M, alpha, beta, Cin, B.DTYPE_F64)
        outs.append(got)
    il = np.tril_indices(N)
    assert np.array_equal(outs[0][il], outs[1][il])


@pytest.mark.parametrize("M", [5, 16, 33, 48])
def test_f64_persistent_form_with_items_of_one_to_three_k_steps(M):
    """Items shorter than the ring of stages (one to three K-steps of 16 columns): the hand-over of the
    accumulators' image between the MMA warps and the write-out warps must not depend on the ring to keep the
    warps of one item together - warps without a tile in an item run ahead.  Long list, ragged edge, repeated."""
    N = 4100
    A = make_A(N, M, B.DTYPE_F64, seed=350 + M, kind="int")
    dA = torch.from_numpy(A).cuda()
    ref, _ = O.syrk_lower(A, None, 1.0, 0.0, B.DTYPE_F64)
    il = np.tril_indices(N)
    try:
        B.syrk_set_f64_launch(B.F64_LAUNCH_PERSISTENT)
        for rep in range(3):
            dC = torch.full((N, N), float("nan"), dtype=torch.float64, device="cuda")
            B.syrk_lower(N, M, dA, M, dC, N, 1.0, 0.0, B.DTYPE_F64)
            torch.cuda.synchronize()
            assert B.syrk_last_status() == 0
            assert np.array_equal(dC.cpu().numpy()[il], ref[il]), rep
    finally:
        B.syrk_set_f64_launch(B.F64_LAUNCH_AUTO)


def test_f64_persistent_form_repeated_and_on_two_streams():
    """The item counter is left at zero by every launch, and each stream has its own: repeated
    calls on one stream and interleaved calls on two streams all give the reference result."""
    import torch
    N, M = 2100, 64
    A = make_A(N, M, B.DTYPE_F64, seed=31, kind="int")
    dA = torch.from_numpy(A).cuda()
    ref, _ = O.syrk_lower(A, None, 1.0, 0.0, B.DTYPE_F64)
    il = np.tril_indices(N)
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    outs = []
    try:
        B.syrk_set_f64_launch(B.F64_LAUNCH_PERSISTENT)
        torch.cuda.synchronize()
        for rep in range(3):
            for s in streams:
                dC = torch.zeros((N, N), dtype=torch.float64, device="cuda")
                s.wait_stream(torch.cuda.current_stream())
                with torch.cuda.stream(s):
                    B.syrk_lower(N, M, dA, M, dC, N, 1.0, 0.0, B.DTYPE_F64, stream=s.cuda_stream)
                outs.append(dC)
        torch.cuda.synchronize()
    finally:
        B.syrk_set_f64_launch(B.F64_LAUNCH_AUTO)
    assert B.syrk_last_status() == 0
    for dC in outs:
        assert np.array_equal(dC.cpu().numpy()[il], ref[il])


def test_f64_call_inside_stream_capture_replays_correctly():
    """During stream capture the library uses the one-block-per-item form (a captured graph may be
    replayed on several streams at once); the replayed graph gives the reference result."""
    import torch
    N, M = 1500, 48
    A = make_A(N, M, B.DTYPE_F64, seed=32, kind="int")
    dA = torch.from_numpy(A).cuda()
    dC = torch.zeros((N, N), dtype=torch.float64, device="cuda")
    B.syrk_lower(N, M, dA, M, dC, N, 1.0, 0.0, B.DTYPE_F64)          # builds the cached work list first
    torch.cuda.synchronize()
    dC.zero_()
    g = torch.cuda.CUDAGraph()
    try:
        B.syrk_set_f64_launch(B.F64_LAUNCH_PERSISTENT)
        with torch.cuda.graph(g):
            B.syrk_lower(N, M, dA, M, dC, N, 1.0, 1.0, B.DTYPE_F64,
                         stream=torch.cuda.current_stream().cuda_stream)
    finally:
        B.syrk_set_f64_launch(B.F64_LAUNCH_AUTO)
    g.replay(); g.replay()
    torch.cuda.synchronize()
    assert B.syrk_last_status() == 0
    ref, _ = O.syrk_lower(A, None, 2.0, 0.0, B.DTYPE_F64)             # two accumulating replays
    il = np.tril_indices(N)
    assert np.array_equal(dC.cpu().numpy()[il], ref[il])


@pytest.mark.parametrize("tn", [False, True], ids=["nxm", "mxn"])
@pytest.mark.parametrize("split", [2, 3, 7])
def test_f64_k_split_forced(split, tn):
    """FP64 K-split: slices of the inner dimension into partial matrices, summed in slice order.
    Ragged last slice and last K-step, ragged N, general alpha / beta, both storage orders; integer
    inputs must still match bit for bit."""
    for n, (N, M) in enumerate([(258, 1030), (1056, 2048), (64, 4099 if not tn else 4100), (700, 528)]):
        A = make_A(N, M, B.DTYPE_F64, seed=900 + n)
        Ai = make_A(N, M, B.DTYPE_F64, seed=950 + n, kind="int")
        Cin = I.random_c(N, 960 + n, B.DTYPE_F64)
        try:
            B.syrk_set_split_k(split)
            got, ref, bound = run_case(A, B.DTYPE_F64, -1.5, 0.5, Cin, tn=tn)
            goti, refi, boundi = run_case(Ai, B.DTYPE_F64, 1.0, 0.0, poison=True, tn=tn)
        finally:
            B.syrk_set_split_k(0)
        assert_within_tolerance(got, ref, bound, M, -1.5, 0.5, Cin, B.DTYPE_F64)
        assert_within_tolerance(goti, refi, boundi, M, 1.0, 0.0, None, B.DTYPE_F64, exact=True)


def test_f64_k_split_automatic_for_short_work_lists():
    """N = 1024 has about 60 work items: with M = 8192 the library cuts the inner dimension by itself."""
    N, M = 1024, 8192
    A = make_A(N, M, B.DTYPE_F64, seed=980)
    Cin = I.random_c(N, 981, B.DTYPE_F64)
    got, ref, bound = run_case(A, B.DTYPE_F64, 1.0, -1.0, Cin, ldc=N + 3)
    assert_within_tolerance(got, ref, bound, M, 1.0, -1.0, Cin, B.DTYPE_F64)


@pytest.mark.parametrize("tn", [False, True], ids=["nxm", "mxn"])
@pytest.mark.parametrize("slices,tail", [(2, 1), (3, 7), (5, 10 ** 6)])
def test_f64_tail_k_split_forced(slices, tail, tn):
    """FP64 tail K-split: the last `tail` items of the list run as `slices` blocks each and a second
    kernel sums their partial tiles in slice order (one item, a few items spanning kinds, every item).
    Triangle blocks with their 16th warp, rectangles and diagonal blocks, ragged N and last K-step,
    general alpha / beta with a pitch, integer inputs bit for bit, and the same bits when repeated."""
    for n, (N, M) in enumerate([(1056, 272), (2100, 130), (700, 1030)]):
        A = make_A(N, M, B.DTYPE_F64, seed=1000 + n)
        Ai = make_A(N, M, B.DTYPE_F64, seed=1050 + n, kind="int")
        Cin = I.random_c(N, 1060 + n, B.DTYPE_F64)
        il = np.tril_indices(N)
        by_form = []
        for form in (B.F64_LAUNCH_PER_ITEM, B.F64_LAUNCH_PERSISTENT):      # blocks per slice / slices as further tickets
            try:
                B.syrk_set_f64_launch(form)
                B.syrk_set_f64_tail_split(slices, tail)
                got, ref, bound = run_case(A, B.DTYPE_F64, -1.5, 0.5, Cin, ldc=N + 2, tn=tn)
                again, _, _ = run_case(A, B.DTYPE_F64, -1.5, 0.5, Cin, ldc=N + 2, tn=tn)
                got1, ref1, bound1 = run_case(A, B.DTYPE_F64, -1.0, 1.0, Cin, tn=tn)
                goti, refi, boundi = run_case(Ai, B.DTYPE_F64, 1.0, 0.0, poison=True, tn=tn)
            finally:
                B.syrk_set_f64_tail_split(0)
                B.syrk_set_f64_launch(B.F64_LAUNCH_AUTO)
            assert_within_tolerance(got, ref, bound, M, -1.5, 0.5, Cin, B.DTYPE_F64)
            assert_within_tolerance(got1, ref1, bound1, M, -1.0, 1.0, Cin, B.DTYPE_F64)
            assert np.array_equal(got[il], again[il])
            assert_within_tolerance(goti, refi, boundi, M, 1.0, 0.0, None, B.DTYPE_F64, exact=True)
            by_form.append((got[il], got1[il]))
        assert np.array_equal(by_form[0][0], by_form[1][0]) and np.array_equal(by_form[0][1], by_form[1][1])


def test_f64_tail_k_split_automatic():
    """A list of a few rounds of long items (3000 x 2048: 319 items of 128 K-steps for 148 SMs): the library
    cuts the tail by itself; switched off, the result agrees within tolerance (another summation order)."""
    N, M = 3000, 2048
    A = make_A(N, M, B.DTYPE_F64, seed=1100)
    Cin = I.random_c(N, 1101, B.DTYPE_F64)
    got, ref, bound = run_case(A, B.DTYPE_F64, 1.0, -1.0, Cin)
    assert_within_tolerance(got, ref, bound, M, 1.0, -1.0, Cin, B.DTYPE_F64)
    try:
        B.syrk_set_f64_tail_split(1)
        off, _, _ = run_case(A, B.DTYPE_F64, 1.0, -1.0, Cin)
    finally:
        B.syrk_set_f64_tail_split(0)
    assert_within_tolerance(off, ref, bound, M, 1.0, -1.0, Cin, B.DTYPE_F64)
    Ai = make_A(N, 1100, B.DTYPE_F64, seed=1102, kind="int")
    goti, refi, boundi = run_case(Ai, B.DTYPE_F64, 1.0, 0.0)
    assert_within_tolerance(goti, refi, boundi, 1100, 1.0, 0.0, None, B.DTYPE_F64, exact=True)


def test_tf32_low_order_bits_of_the_inputs_are_ignored():
    """The tensor core reads the 19 high-order bits of every binary32 input.  With values whose
    low 13 bits are set the result must equal, bit for bit, the result for the same values with
    those bits cleared (all products and sums below are exact in binary32)."""
    N, M = 300, 64
    rng = np.random.default_rng(77)
    base = rng.integers(-2, 3, size=(N, M)).astype(np.float32)             # exact in TF32
    noise = (rng.integers(1, 1 << 13, size=(N, M)).astype(np.uint32))      # only bits 0..12
    dirty = (base.view(np.uint32) | np.where(base != 0, noise, 0).astype(np.uint32)).view(np.float32)
    assert np.array_equal(I.f32_keep_tf32_bits(dirty), base) and not np.array_equal(dirty, base)
    got_dirty, ref, bound = run_case(dirty, B.DTYPE_TF32_F32, 1.0, 0.0)
    got_clean, _, _ = run_case(base, B.DTYPE_TF32_F32, 1.0, 0.0)
    il = np.tril_indices(N)
    assert np.array_equal(got_dirty[il], got_clean[il])
    assert np.array_equal(got_dirty[il], ref[il])                           # the reference drops them too
    # the plain-load path (unaligned A) makes the same reading
    got_plain, _, _ = run_case(dirty, B.DTYPE_TF32_F32, 1.0, 0.0, lda=M + 3, a_offset=1)
    assert np.array_equal(got_plain[il], ref[il])


@DT
def test_host_buffer_entry_point_pipelined_blocks(dtype):
    """Inputs large enough for the host entry point to upload A in several column blocks and to
    bring C back in bands (A > 64 MB), with beta != 0, a ragged last block and host pitches."""
    N, M = {B.DTYPE_F64: (1500, 9000), B.DTYPE_BF16_F32: (2304, 24000), B.DTYPE_TF32_F32: (1800, 12100),
            B.DTYPE_E4M3_F32: (2304, 48000), B.DTYPE_F16_F32: (2304, 24000)}[dtype]
    A = make_A(N, M, dtype, seed=51)
    lda, ldc = M + 16, N + 5
    Abig = np.zeros((N, lda), dtype=A.dtype)
    Abig[:, :M] = A
    Cin = I.random_c(N, 52, dtype, ldc)
    C = Cin.copy()
    B.syrk_lower_host(N, M, Abig, lda, C, ldc, 0.5, -1.0, dtype)
    ii, jj = np.tril_indices(N)
    pick = np.random.default_rng(53).choice(ii.size, size=20000, replace=False)
    ii, jj = ii[pick], jj[pick]
    ref, bound = O.syrk_entries(ii, jj, A, None, 0.5, 0.0, dtype)
    ref = ref - Cin[ii, jj].astype(np.float64)
    tol = O.tolerance(M, bound, np.abs(Cin[ii, jj]), 0.5, -1.0, dtype)
    assert np.all(np.abs(C[ii, jj].astype(np.float64) - ref) <= tol)
    iu = np.triu_indices(N, 1)
    assert np.array_equal(C[:, :N][iu], Cin[:, :N][iu])           # strict upper triangle untouched
    assert np.array_equal(C[:, N:], Cin[:, N:])                   # and the padding columns


@DT
def test_host_buffer_entry_point_row_band_pipeline(dtype):
    """Page-locked host buffers and N >= 4096: the entry point uploads A, computes and downloads C
    band of rows by band of rows.  Ragged N, pitches, beta != 0; sampled entries plus every entry
    next to the band and tile boundaries of a few rows; upper triangle and padding untouched."""
    import torch
    N, M = {B.DTYPE_F64: (4100, 200), B.DTYPE_BF16_F32: (4500, 520), B.DTYPE_TF32_F32: (4230, 260),
            B.DTYPE_E4M3_F32: (4400, 1040), B.DTYPE_F16_F32: (4500, 520)}[dtype]
    A = make_A(N, M, dtype, seed=71)
    lda, ldc = M + 32, N + 6
    Abig = np.zeros((N, lda), dtype=A.dtype)
    Abig[:, :M] = A
    Cin = I.random_c(N, 72, dtype, ldc)
    hA = torch.from_numpy(Abig.view(np.int16) if Abig.dtype == np.uint16 else Abig).pin_memory()
    hC = torch.from_numpy(Cin.copy()).pin_memory()
    for alpha, beta in ((0.5, -1.0), (1.0, 0.0)):
        hC.copy_(torch.from_numpy(Cin))
        B.syrk_lower_host(N, M, hA, lda, hC, ldc, alpha, beta, dtype)
        C = hC.numpy()
        rng = np.random.default_rng(73)
        ii = rng.integers(0, N, size=30000)
        jj = (rng.random(30000) * (ii + 1)).astype(np.int64)
        rows = np.array([0, 127, 128, 255, 256, 257, 511, 512, 2047, 2048, 4095, 4096, N - 1])
        rows = rows[rows < N]
        ii = np.concatenate([ii] + [np.full(r + 1, r) for r in rows])
        jj = np.concatenate([jj] + [np.arange(r + 1) for r in rows])
        ref, bound = O.syrk_entries(ii, jj, A, None, alpha, 0.0, dtype)
        ref = ref + beta * Cin[ii, jj].astype(np.float64)
        tol = O.tolerance(M, bound, np.abs(Cin[ii, jj]), alpha, beta, dtype)
        assert np.all(np.abs(C[ii, jj].astype(np.float64) - ref) <= tol)
        iu = np.triu_indices(N, 1)
        assert np.array_equal(C[:, :N][iu], Cin[:, :N][iu])
        assert np.array_equal(C[:, N:], Cin[:, N:])


@pytest.mark.parametrize("dtype", [B.DTYPE_F64, B.DTYPE_BF16_F32, B.DTYPE_E4M3_F32], ids=["f64", "bf16", "e4m3"])
def test_host_buffer_entry_point_column_block_pipeline_with_page_locked_buffers(dtype):
    """The same page-locked call as above with the column-block pipeline forced: A goes up in blocks of
    columns, each block's update runs the device call's schedule (triangle blocks here: the file pins them)
    while the next block travels, C comes down in bands afterwards.  A wide operand (several blocks, ragged
    last one), ragged N, pitches, beta != 0; sampled entries plus whole rows at band and tile boundaries."""
    import torch
    N, M = {B.DTYPE_F64: (4100, 2300), B.DTYPE_BF16_F32: (4500, 9000), B.DTYPE_E4M3_F32: (4400, 17000)}[dtype]
    assert B.syrk_host_pipeline_for(N, M, True) == B.HOST_ROW_BANDS and B.syrk_host_pipeline_for(N, M, False) == B.HOST_COLUMN_BLOCKS
    A = make_A(N, M, dtype, seed=81)
    lda, ldc = M + 32, N + 6
    Abig = np.zeros((N, lda), dtype=A.dtype)
    Abig[:, :M] = A
    Cin = I.random_c(N, 82, dtype, ldc)
    hA = torch.from_numpy(Abig.view(np.int16) if Abig.dtype == np.uint16 else Abig).pin_memory()
    hC = torch.from_numpy(Cin.copy()).pin_memory()
    alpha, beta = 0.5, -1.0
    try:
        B.syrk_set_host_pipeline(B.HOST_COLUMN_BLOCKS)
        assert B.syrk_host_pipeline_for(N, M, True) == B.HOST_COLUMN_BLOCKS
        B.syrk_lower_host(N, M, hA, lda, hC, ldc, alpha, beta, dtype)
    finally:
        B.syrk_set_host_pipeline(B.HOST_AUTO)
    C = hC.numpy()
    rng = np.random.default_rng(83)
    ii = rng.integers(0, N, size=20000)
    jj = (rng.random(20000) * (ii + 1)).astype(np.int64)
    rows = np.array([0, 127, 128, 255, 256, 2047, 2048, 4095, 4096, N - 1])
    rows = rows[rows < N]
    ii = np.concatenate([ii] + [np.full(r + 1, r) for r in rows])
    jj = np.concatenate([jj] + [np.arange(r + 1) for r in rows])
    ref, bound = O.syrk_entries(ii, jj, A, None, alpha, 0.0, dtype)
    ref = ref + beta * Cin[ii, jj].astype(np.float64)
    tol = O.tolerance(M, bound, np.abs(Cin[ii, jj]), alpha, beta, dtype)
    assert np.all(np.abs(C[ii, jj].astype(np.float64) - ref) <= tol)
    iu = np.triu_indices(N, 1)
    assert np.array_equal(C[:, :N][iu], Cin[:, :N][iu])
    assert np.array_equal(C[:, N:], Cin[:, N:])
    with pytest.raises(B.SyrkError):
        B.syrk_set_host_pipeline(7)
