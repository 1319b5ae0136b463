"""GPU parity at the full benchmark sizes, in the launch configuration bench.py times.

Where the whole triangle is too slow for the CPU reference, sampled entries are
checked one by one: uniformly random pairs (i >= j), every diagonal entry of a few
tiles, and entries on tile-boundary rows and columns.  Tolerances as in
test_gpu_syrk.py.
"""
import numpy as np
import pytest
import torch

from oracle import syrk as O
from paper_2202_10217_b200 import binding as B
from paper_2202_10217_b200 import inputs as I

pytestmark = pytest.mark.gpu


def upload_A(A, dtype):
    if dtype in (B.DTYPE_F64, B.DTYPE_TF32_F32, B.DTYPE_E4M3_F32):
        return torch.from_numpy(A).cuda()
    return torch.from_numpy(A.view(np.int16)).cuda().view(torch.float16 if dtype == B.DTYPE_F16_F32 else torch.bfloat16)


def sample_pairs(N, count, tile, seed):
    rng = np.random.default_rng(seed)
    i = rng.integers(0, N, size=count)
    j = (rng.random(count) * (i + 1)).astype(np.int64)
    extra_i, extra_j = [], []
    edges = sorted({0, N - 1, tile - 1, tile, N // 2, (N // tile) * tile - 1, max((N // tile) * tile - tile, 0)})
    for r in edges:
        if 0 <= r < N:
            cols = np.unique(np.clip(np.array([0, r, r - 1, r // 2, (r // tile) * tile, (r // tile) * tile - 1]), 0, r))
            extra_i += [r] * len(cols)
            extra_j += list(cols)
    d = np.arange(0, min(N, 4 * tile))                    # diagonal entries of the first tiles
    extra_i += list(d) + list(N - 1 - d)
    extra_j += list(d) + list(N - 1 - d)
    return np.concatenate([i, np.array(extra_i, dtype=np.int64)]), np.concatenate([j, np.array(extra_j, dtype=np.int64)])


def check_sampled(dC, Cin_vals, A, wl, ii, jj):
    got = dC[torch.from_numpy(ii).cuda(), torch.from_numpy(jj).cuda()].cpu().numpy().astype(np.float64)
    ref, bound = O.syrk_entries(ii, jj, A, None, wl.alpha, 0.0, wl.dtype)
    if wl.beta != 0.0:
        ref = ref + wl.beta * Cin_vals
    tol = O.tolerance(wl.M, bound, None if Cin_vals is None else np.abs(Cin_vals), wl.alpha, wl.beta, wl.dtype)
    err = np.abs(got - ref)
    assert np.all(err <= tol), "%d sampled entries out of tolerance (worst ratio %.3g)" % (
        int((err > tol).sum()), float(np.max(err / np.maximum(tol, 1e-300))))
    return float(np.max(err / np.maximum(tol, 1e-300)))


def run_config(key, samples, gram=False):
    """`gram`: the same operand handed over stored M x N, through syrk_lower_tn."""
    wl = I.CONFIGS[key]
    A = wl.make_A()
    dA = upload_A(A, wl.dtype)
    sentinel = float("nan")
    dC = torch.full((wl.N, wl.N), sentinel, dtype=torch.float64 if wl.dtype == B.DTYPE_F64 else torch.float32,
                    device="cuda")
    if gram:
        dA = dA.t().contiguous()
        B.syrk_lower_tn(wl.N, wl.M, dA, wl.N, dC, wl.N, wl.alpha, wl.beta, wl.dtype)
    else:
        B.syrk_lower(wl.N, wl.M, dA, wl.M, dC, wl.N, wl.alpha, wl.beta, wl.dtype)
    torch.cuda.synchronize()
    assert B.syrk_last_status() == 0
    # strict upper triangle untouched (still NaN), lower triangle fully written
    nan_mask = torch.isnan(dC)
    assert bool(torch.equal(nan_mask, torch.triu(torch.ones_like(nan_mask), diagonal=1)))
    return wl, A, dC


def test_config1_full_triangle():
    wl, A, dC = run_config("c1", 0)
    ref, bound = O.syrk_lower(A, None, wl.alpha, 0.0, wl.dtype)
    il = np.tril_indices(wl.N)
    got = dC.cpu().numpy()
    assert np.all(np.abs(got[il] - ref[il]) <= O.tolerance(wl.M, bound[il], None, 1.0, 0.0, wl.dtype))


def test_config2_full_triangle():
    wl, A, dC = run_config("c2", 0)
    ref, bound = O.syrk_lower(A, None, wl.alpha, 0.0, wl.dtype)
    il = np.tril_indices(wl.N)
    got = dC.cpu().numpy()
    assert np.all(np.abs(got[il] - ref[il]) <= O.tolerance(wl.M, bound[il], None, 1.0, 0.0, wl.dtype))


def test_config2_gram_form_full_triangle():
    wl, A, dC = run_config("c2", 0, gram=True)
    ref, bound = O.syrk_lower(A, None, wl.alpha, 0.0, wl.dtype)
    il = np.tril_indices(wl.N)
    got = dC.cpu().numpy()
    assert np.all(np.abs(got[il] - ref[il]) <= O.tolerance(wl.M, bound[il], None, 1.0, 0.0, wl.dtype))


def test_config3_gram_form_sampled():
    wl, A, dC = run_config("c3", 1 << 20, gram=True)
    ii, jj = sample_pairs(wl.N, 1 << 20, 128, seed=35)
    check_sampled(dC, None, A, wl, ii, jj)


def test_config4_gram_form_sampled_split_k():
    wl, A, dC = run_config("c4", 1 << 14, gram=True)
    ii, jj = sample_pairs(wl.N, 1 << 14, 128, seed=45)
    check_sampled(dC, None, A, wl, ii, jj)


def test_config3_sampled():
    wl, A, dC = run_config("c3", 1 << 20)
    ii, jj = sample_pairs(wl.N, 1 << 20, 128, seed=33)
    check_sampled(dC, None, A, wl, ii, jj)


def test_config4_sampled_split_k():
    wl, A, dC = run_config("c4", 1 << 14)
    ii, jj = sample_pairs(wl.N, 1 << 14, 128, seed=44)
    check_sampled(dC, None, A, wl, ii, jj)
    # run-to-run bitwise reproducibility of the K-split reduction
    dA = upload_A(A, wl.dtype)
    dC2 = torch.zeros_like(dC)
    B.syrk_lower(wl.N, wl.M, dA, wl.M, dC2, wl.N, wl.alpha, wl.beta, wl.dtype)
    torch.cuda.synchronize()
    il = torch.tril_indices(wl.N, wl.N, device="cuda")
    assert torch.equal(dC[il[0], il[1]], dC2[il[0], il[1]])


def test_config5_trailing_update_sweep():
    """C_n <- C_n - A_n A_n^T on the trailing n x n view of one 32768^2 matrix
    (n*I + G G^T / 512), n = 32768, 32256, ..., 512: 64 calls with ldc = 32768."""
    n_max, step = 32768, 512
    G = torch.from_numpy(I.sweep_factor(n_max)).cuda()
    C = torch.matmul(G, G.T) / float(I.SWEEP_K)                       # input preparation
    C.diagonal().add_(float(n_max))
    del G
    worst = 0.0
    for n in I.sweep_sizes(n_max, step):
        A = I.sweep_panel(n, n_max)
        dA = torch.from_numpy(A).cuda()
        off = n_max - n
        view_ptr = C.data_ptr() + (off * n_max + off) * 8
        ii, jj = sample_pairs(n, 2048, 32, seed=500 + n // step)
        gi, gj = torch.from_numpy(ii + off).cuda(), torch.from_numpy(jj + off).cuda()
        before = C[gi, gj].cpu().numpy()
        upper_probe = C[gj[:64], gi[:64]].clone()                     # (j, i): above or on the diagonal
        B.syrk_lower(n, I.SWEEP_K, dA, I.SWEEP_K, view_ptr, n_max, -1.0, 1.0, B.DTYPE_F64)
        torch.cuda.synchronize()
        assert B.syrk_last_status() == 0
        got = C[gi, gj].cpu().numpy()
        ref, bound = O.syrk_entries(ii, jj, A, None, -1.0, 0.0, B.DTYPE_F64)
        ref = ref + before
        tol = O.tolerance(I.SWEEP_K, bound, np.abs(before), -1.0, 1.0, B.DTYPE_F64)
        err = np.abs(got - ref)
        assert np.all(err <= tol), "n=%d: %d entries out of tolerance" % (n, int((err > tol).sum()))
        worst = max(worst, float(np.max(err / tol)))
        strict = (ii[:64] != jj[:64])
        assert torch.equal(C[gj[:64], gi[:64]][torch.from_numpy(strict).cuda()],
                           upper_probe[torch.from_numpy(strict).cuda()]), "upper triangle touched"
    assert worst <= 1.0


@pytest.mark.parametrize("split", [2, 3, 7])
def test_forced_split_k_matches_reference(split):
    N, M = 700, 1280
    A = I.small_int_bf16(N, M, seed=split)
    Cin = (np.random.default_rng(1).integers(-4, 5, size=(N, N))).astype(np.float32)
    dA = upload_A(A, B.DTYPE_BF16_F32)
    dC = torch.from_numpy(Cin.copy()).cuda()
    try:
        B.syrk_set_split_k(split)
        B.syrk_lower(N, M, dA, M, dC, N, 2.0, -1.0, B.DTYPE_BF16_F32)
        torch.cuda.synchronize()
    finally:
        B.syrk_set_split_k(0)
    assert B.syrk_last_status() == 0
    ref, _ = O.syrk_lower(A, Cin, 2.0, -1.0, B.DTYPE_BF16_F32)
    got = dC.cpu().numpy().astype(np.float64)
    il, iu = np.tril_indices(N), np.triu_indices(N, 1)
    assert np.array_equal(got[il], ref[il])                          # integers: exact in any order
    assert np.array_equal(got[iu], Cin[iu].astype(np.float64))


@pytest.mark.parametrize("dtype,N,M", [(B.DTYPE_BF16_F32, 20001, 104), (B.DTYPE_F64, 12003, 50),
                                       (B.DTYPE_TF32_F32, 16384, 4096), (B.DTYPE_TF32_F32, 20001, 52),
                                       (B.DTYPE_E4M3_F32, 16384, 8192), (B.DTYPE_E4M3_F32, 20001, 208),
                                       (B.DTYPE_F16_F32, 16384, 4096), (B.DTYPE_F16_F32, 20001, 104)])
def test_large_ragged_sizes_sampled(dtype, N, M):
    """Hundreds of tile rows with a ragged last tile and a ragged last K-step; alpha/beta general."""
    A = {B.DTYPE_F64: I.normal_f64, B.DTYPE_BF16_F32: I.normal_bf16, B.DTYPE_TF32_F32: I.normal_f32,
         B.DTYPE_E4M3_F32: I.normal_e4m3, B.DTYPE_F16_F32: I.normal_f16}[dtype](N, M, 77)
    dA = upload_A(A, dtype)
    tdt = torch.float64 if dtype == B.DTYPE_F64 else torch.float32
    gen = torch.Generator(device="cuda").manual_seed(5)
    dC = torch.randn((N, N), dtype=tdt, device="cuda", generator=gen)
    ii, jj = sample_pairs(N, 1 << 16, 32 if dtype == B.DTYPE_F64 else 128, seed=78)
    gi, gj = torch.from_numpy(ii).cuda(), torch.from_numpy(jj).cuda()
    before = dC[gi, gj].cpu().numpy().astype(np.float64)
    up_before = dC[gj[:256], gi[:256]].clone()
    alpha, beta = 0.75, -1.25
    B.syrk_lower(N, M, dA, M, dC, N, alpha, beta, dtype)
    torch.cuda.synchronize()
    assert B.syrk_last_status() == 0
    got = dC[gi, gj].cpu().numpy().astype(np.float64)
    ref, bound = O.syrk_entries(ii, jj, A, None, alpha, 0.0, dtype)
    ref = ref + beta * before
    tol = O.tolerance(M, bound, np.abs(before), alpha, beta, dtype)
    assert np.all(np.abs(got - ref) <= tol)
    strict = torch.from_numpy(ii[:256] != jj[:256]).cuda()
    assert torch.equal(dC[gj[:256], gi[:256]][strict], up_before[strict])
