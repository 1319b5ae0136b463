"""The failure path of the bounded waits, on the GPU without a fault: a self-test kernel waits on a barrier
that nothing arrives on; its wait runs out after the library's time limit (about two seconds), the kernel
returns normally, the host reads the status once, and the context is as usable as before."""
import time

import numpy as np
import pytest
import torch

from paper_2202_10217_b200 import binding as B
from paper_2202_10217_b200 import inputs as I

from gpu_util import assert_within_tolerance, run_case

pytestmark = pytest.mark.gpu


def test_a_wait_that_runs_out_is_reported_once_and_the_context_stays_usable():
    torch.cuda.synchronize()
    assert B.syrk_last_status() == 0
    t0 = time.perf_counter()
    B.syrk_selftest_bounded_wait()
    torch.cuda.synchronize()                       # the kernel ends by itself when its wait gives up
    waited = time.perf_counter() - t0
    assert 1.0 < waited < 10.0
    assert B.syrk_last_status() == -8              # SYRK_ERR_DEVICE_WAIT, reported ...
    assert B.strerror(-8) == "a bounded wait inside a kernel ran out"
    assert B.syrk_last_status() == 0               # ... once
    for dtype, N, M in [(B.DTYPE_F64, 300, 40), (B.DTYPE_BF16_F32, 300, 72)]:
        A = I.normal_f64(N, M, 8000) if dtype == B.DTYPE_F64 else I.normal_bf16(N, M, 8001)
        got, ref, bound = run_case(A, dtype, 1.0, 0.0)
        assert_within_tolerance(got, ref, bound, M, 1.0, 0.0, None, dtype)
