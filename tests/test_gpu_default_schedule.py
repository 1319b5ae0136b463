"""GPU parity of what the library does by default (SYRK_SCHEDULE_AUTO) and of its per-stream state.

* The schedules the automatic rule selects, at the full benchmark sizes, against the CPU reference on
  sampled entries: config 4 (2048 x 262144) on square blocks on CTA pairs with a K-split, config 3
  (16384 x 4096) on triangle blocks; and the other way round under explicit settings (config 3 on the
  pair schedule, config 4 on triangle blocks), so that every kernel is checked at both sizes.
* K-split calls on two streams at once (each stream has its own workspace) on disjoint outputs.
* The status word is per stream.
* A K-split call inside stream capture after syrk_plan_prepare_stream; refusal when it would allocate.
"""
import numpy as np
import pytest
import torch

from oracle import syrk as O
from paper_2202_10217_b200 import binding as B
from paper_2202_10217_b200 import inputs as I

from test_gpu_configs import check_sampled, sample_pairs, upload_A
from test_gpu_syrk import make_A

pytestmark = pytest.mark.gpu


def run_full_size(key, schedule):
    wl = I.CONFIGS[key]
    A = wl.make_A()
    dA = upload_A(A, wl.dtype)
    dC = torch.full((wl.N, wl.N), float("nan"), dtype=torch.float32, device="cuda")
    try:
        B.syrk_set_schedule(schedule)
        B.syrk_lower(wl.N, wl.M, dA, wl.M, dC, wl.N, wl.alpha, wl.beta, wl.dtype)
        torch.cuda.synchronize()
    finally:
        B.syrk_set_schedule(B.SCHEDULE_DEFAULT)
    assert B.syrk_last_status() == 0
    nan_mask = torch.isnan(dC)                         # strict upper triangle untouched, lower fully written
    assert bool(torch.equal(nan_mask, torch.triu(torch.ones_like(nan_mask), diagonal=1)))
    return wl, A, dC


@pytest.mark.parametrize("key,schedule,runs", [
    ("c4", B.SCHEDULE_DEFAULT, B.SCHEDULE_PAIR_SQUARE),        # what the rule picks for a 55-item list
    ("c3", B.SCHEDULE_DEFAULT, B.SCHEDULE_TBS),                # 2848 items: triangle blocks
    ("c3", B.SCHEDULE_PAIR_SQUARE, B.SCHEDULE_PAIR_SQUARE),
    ("c4", B.SCHEDULE_TBS, B.SCHEDULE_TBS),                    # triangle blocks in eight K-slices
], ids=["c4-default", "c3-default", "c3-pair", "c4-tbs"])
def test_full_size_configs_under_each_schedule(key, schedule, runs):
    wl = I.CONFIGS[key]
    try:
        B.syrk_set_schedule(schedule)
        assert B.syrk_effective_schedule(wl.N, wl.M, wl.dtype) == runs
    finally:
        B.syrk_set_schedule(B.SCHEDULE_DEFAULT)
    wl, A, dC = run_full_size(key, schedule)
    count = 1 << (20 if key == "c3" else 14)           # config 4: 262144 products per sampled entry
    ii, jj = sample_pairs(wl.N, count, 128, seed=91)
    check_sampled(dC, None, A, wl, ii, jj)


@pytest.mark.parametrize("dtype,N,M,schedule", [
    (B.DTYPE_BF16_F32, 1408, 8192, B.SCHEDULE_TBS),            # tcgen05 triangle-block kernel, forced slices
    (B.DTYPE_BF16_F32, 2048, 8192, B.SCHEDULE_PAIR_SQUARE),    # CTA-pair kernel, its own K-split
    (B.DTYPE_F64, 1024, 4096, B.SCHEDULE_TBS),                 # FP64 kernel, partial matrices
], ids=["tcgen05-tbs", "pair", "f64"])
def test_k_split_calls_on_two_streams_at_once(dtype, N, M, schedule):
    """Two streams, each running K-split calls on its own C from its own A, enqueued alternately without
    any synchronisation in between: the partial tiles of one must not end up in the other's sum.
    Integer inputs: every result must equal the reference bit for bit."""
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    As = [make_A(N, M, dtype, seed=8100 + s, kind="int") for s in range(2)]
    dAs = [upload_A(A, dtype) for A in As]
    cdt = torch.float64 if dtype == B.DTYPE_F64 else torch.float32
    outs = [[torch.zeros((N, N), dtype=cdt, device="cuda") for _ in range(3)] for _ in range(2)]
    torch.cuda.synchronize()
    try:
        B.syrk_set_schedule(schedule)
        B.syrk_set_split_k(4)
        for rep in range(3):
            for s, st in enumerate(streams):
                B.syrk_lower(N, M, dAs[s], M, outs[s][rep], N, 1.0, 0.0, dtype, stream=st.cuda_stream)
        torch.cuda.synchronize()
    finally:
        B.syrk_set_split_k(0)
        B.syrk_set_schedule(B.SCHEDULE_DEFAULT)
    for st in streams:
        assert B.syrk_last_status(st.cuda_stream) == 0
    il = np.tril_indices(N)
    for s in range(2):
        ref, _ = O.syrk_lower(As[s], None, 1.0, 0.0, dtype)
        for rep in range(3):
            assert np.array_equal(outs[s][rep].cpu().numpy().astype(np.float64)[il], ref[il]), (s, rep)


def test_status_word_is_per_stream():
    """A wait that runs out on one stream (the library's self-test kernel, about two seconds) is reported
    for that stream and for the all-streams query, not for another stream; and it is reported once."""
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    N, M = 300, 64
    A = make_A(N, M, B.DTYPE_F64, seed=8200, kind="int")
    dA = upload_A(A, B.DTYPE_F64)
    dC = torch.zeros((N, N), dtype=torch.float64, device="cuda")
    torch.cuda.synchronize()
    B.syrk_selftest_bounded_wait(s1.cuda_stream)
    B.syrk_lower(N, M, dA, M, dC, N, 1.0, 0.0, B.DTYPE_F64, stream=s2.cuda_stream)
    torch.cuda.synchronize()
    assert B.syrk_last_status(s2.cuda_stream) == 0
    assert B.syrk_last_status(s1.cuda_stream) == -8
    assert B.syrk_last_status(s1.cuda_stream) == 0
    assert B.syrk_last_status() == 0
    B.syrk_selftest_bounded_wait(s1.cuda_stream)
    torch.cuda.synchronize()
    assert B.syrk_last_status() == -8                      # stream 0 asks for every stream
    assert B.syrk_last_status(s1.cuda_stream) == 0
    ref, _ = O.syrk_lower(A, None, 1.0, 0.0, B.DTYPE_F64)
    il = np.tril_indices(N)
    assert np.array_equal(dC.cpu().numpy()[il], ref[il])


def test_k_split_call_inside_stream_capture_needs_a_prepared_workspace():
    """During capture the library must not allocate (growing a workspace frees the old one, which
    synchronises the device): a K-split call on a stream whose workspace is too small is refused with
    SYRK_ERR_ALLOC and enqueues nothing; after syrk_plan_prepare_stream the same call is captured and the
    replayed graph gives the reference result."""
    N, M = 1536, 16384                                    # 12 tile rows: the default rule takes pairs and cuts K
    assert B.syrk_effective_schedule(N, M, B.DTYPE_BF16_F32) == B.SCHEDULE_PAIR_SQUARE
    A = make_A(N, M, B.DTYPE_BF16_F32, seed=8300, kind="int")
    dA = upload_A(A, B.DTYPE_BF16_F32)
    dC = torch.zeros((N, N), dtype=torch.float32, device="cuda")
    side = torch.cuda.Stream()
    # work lists and a workspace that is too small for the call below (a shorter inner dimension, fewer slices)
    B.syrk_plan_prepare_stream(N, 1024, B.DTYPE_BF16_F32, side.cuda_stream)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        dC.mul_(1.0)                                       # so that the graph is not empty
        with pytest.raises(B.SyrkError) as e:
            B.syrk_lower(N, M, dA, M, dC, N, 1.0, 0.0, B.DTYPE_BF16_F32, stream=side.cuda_stream)
        assert e.value.code == -5
    del g
    torch.cuda.synchronize()
    B.syrk_plan_prepare_stream(N, M, B.DTYPE_BF16_F32, side.cuda_stream)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        B.syrk_lower(N, M, dA, M, dC, N, 1.0, 1.0, B.DTYPE_BF16_F32, stream=side.cuda_stream)
    g.replay(); g.replay()
    torch.cuda.synchronize()
    assert B.syrk_last_status() == 0
    ref, _ = O.syrk_lower(A, None, 2.0, 0.0, B.DTYPE_BF16_F32)        # two accumulating replays
    il = np.tril_indices(N)
    assert np.array_equal(dC.cpu().numpy().astype(np.float64)[il], ref[il])


@pytest.mark.parametrize("pinned", [False, True], ids=["pageable", "page-locked"])
def test_host_buffer_entry_point_under_the_default_schedule(pinned):
    """syrk_lower_host with a short-and-wide BF16 operand: below the band pipeline's size the call uploads A
    in blocks of columns and runs each block through the device call, which under the default rule means
    square blocks on CTA pairs with their own K-split; beta != 0, pitches, ragged last block."""
    N, M = 2304, 24000
    assert B.syrk_effective_schedule(N, M, B.DTYPE_BF16_F32) == B.SCHEDULE_PAIR_SQUARE
    assert B.syrk_host_pipeline_for(N, M, pinned) == B.HOST_COLUMN_BLOCKS
    A = make_A(N, M, B.DTYPE_BF16_F32, seed=8400)
    lda, ldc = M + 16, N + 5
    Abig = np.zeros((N, lda), dtype=A.dtype)
    Abig[:, :M] = A
    Cin = I.random_c(N, 8401, B.DTYPE_BF16_F32, ldc)
    hA = torch.from_numpy(Abig.view(np.int16))
    hC = torch.from_numpy(Cin.copy())
    if pinned:
        hA, hC = hA.pin_memory(), hC.pin_memory()
    B.syrk_lower_host(N, M, hA, lda, hC, ldc, 0.5, -1.0, B.DTYPE_BF16_F32)
    C = hC.numpy()
    ii, jj = np.tril_indices(N)
    pick = np.random.default_rng(8402).choice(ii.size, size=20000, replace=False)
    ii, jj = ii[pick], jj[pick]
    ref, bound = O.syrk_entries(ii, jj, A, None, 0.5, 0.0, B.DTYPE_BF16_F32)
    ref = ref - Cin[ii, jj].astype(np.float64)
    tol = O.tolerance(M, bound, np.abs(Cin[ii, jj]), 0.5, -1.0, B.DTYPE_BF16_F32)
    assert np.all(np.abs(C[ii, jj].astype(np.float64) - ref) <= tol)
    iu = np.triu_indices(N, 1)
    assert np.array_equal(C[:, :N][iu], Cin[:, :N][iu]) and np.array_equal(C[:, N:], Cin[:, N:])
