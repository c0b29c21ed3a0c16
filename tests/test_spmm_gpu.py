"""GPU parity: CSR SpMM through the C ABI against the CPU oracle."""
import numpy as np
import pytest

import gen
import oracle
import paper_2603_07169_b200 as b200sp
from gpu_util import assert_within, run_spmm, store

pytestmark = pytest.mark.gpu

DTYPES = ["f32", "bf16"]


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("k", [1, 3, 8, 17, 32, 64, 100, 256, 264])
def test_small_random_all_k(k, dtype):
    rng = np.random.default_rng(k)
    m, n = 1500, 333
    lens = rng.integers(0, 40, m)
    lens[5] = 3000
    lens[6] = 0
    A = gen.random_csr(m, n, lens, seed=k)
    B = rng.standard_normal(n * k).astype(np.float32)
    Y0 = rng.standard_normal(m * k).astype(np.float32)
    Y, Y_ref, S = run_spmm(A, B, k, None, 1.0, 0.0, dtype)
    assert_within(Y, Y_ref, S, dtype, what="k=%d %s" % (k, dtype))
    Y, Y_ref, S = run_spmm(A, B, k, Y0, 0.5, -2.0, dtype)
    y0f = Y0 if dtype == "f32" else gen.bf16_to_f32(gen.to_bf16(Y0))
    assert_within(Y, Y_ref, S, dtype, 1.0, np.abs(2.0 * y0f.astype(np.float64)).reshape(m, k), what="k=%d %s ab" % (k, dtype))


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("sliced", [0, 1])
def test_long_rows_and_both_kernels(sliced, dtype):
    """Rows above and below the long-row threshold (1024), with the k-sliced and the one-pass kernel."""
    b200sp.b200sp_set_option("spmm_sliced", sliced)
    try:
        rng = np.random.default_rng(3)
        lens = np.array([1024, 1025, 0, 5000, 3, 1023, 20000] + [7] * 300)
        A = gen.random_csr(len(lens), 900, lens, seed=11)
        for k in (8, 64, 72, 256):
            B = rng.standard_normal(900 * k).astype(np.float32)
            Y0 = rng.standard_normal(len(lens) * k).astype(np.float32)
            Y, Y_ref, S = run_spmm(A, B, k, None, 1.0, 0.0, dtype)
            assert_within(Y, Y_ref, S, dtype, what="long rows k=%d" % k)
            Y, Y_ref, S = run_spmm(A, B, k, Y0, -1.0, 0.5, dtype)
            y0f = Y0 if dtype == "f32" else gen.bf16_to_f32(gen.to_bf16(Y0))
            assert_within(Y, Y_ref, S, dtype, 1.0, np.abs(0.5 * y0f.astype(np.float64)).reshape(len(lens), k), what="long rows ab k=%d" % k)
    finally:
        b200sp.b200sp_set_option("spmm_sliced", 1)


@pytest.mark.parametrize("k", [64, 256])
def test_longest_sequential_rows_positive_data(k):
    """Rows of exactly 1024 nonzeros are the longest that one lane group adds in sequence; with all-positive data nothing
    cancels, so this is the case that comes closest to the FP32 bound (chain bound 1024 * 2^-24 * S; measured 0.2-0.25 of 1e-5 * S)."""
    rng = np.random.default_rng(5)
    A = gen.random_csr(400, 4000, np.full(400, 1024), seed=1024)
    A.vals[:] = rng.random(A.nnz).astype(np.float32) + 0.01
    B = rng.random(4000 * k).astype(np.float32) + 0.01
    Y, Y_ref, S = run_spmm(A, B, k, None, 1.0, 0.0, "f32")
    assert assert_within(Y, Y_ref, S, "f32", what="1024-term rows, positive data") < 0.5


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("n,k", [(2048, 4096), (2048, 40), (1500, 72), (300, 264), (5000, 64), (100, 8)])
def test_b_slice_in_shared_memory(n, k, dtype):
    """Few columns: the kernel that holds a slice of B in shared memory (the paper's SpMM shape is n = 2048, K = 4096).
    Covers all three slice widths, n not a multiple of the copy box, k not a multiple of the slice, long rows, beta != 0."""
    rng = np.random.default_rng(n + k)
    m = 3000
    lens = rng.integers(0, 40, m)
    lens[7] = min(n, 2500)
    lens[8] = 0
    A = gen.random_csr(m, n, lens, seed=n)
    B = rng.standard_normal(n * k).astype(np.float32)
    Y0 = rng.standard_normal(m * k).astype(np.float32)
    Y, Y_ref, S = run_spmm(A, B, k, None, 1.0, 0.0, dtype)
    assert_within(Y, Y_ref, S, dtype, what="bstage n=%d k=%d" % (n, k))
    Y, Y_ref, S = run_spmm(A, B, k, Y0, 2.0, -0.5, dtype)
    y0f = Y0 if dtype == "f32" else gen.bf16_to_f32(gen.to_bf16(Y0))
    assert_within(Y, Y_ref, S, dtype, 2.0, np.abs(0.5 * y0f.astype(np.float64)).reshape(m, k), what="bstage ab n=%d k=%d" % (n, k))
    b200sp.b200sp_check()


@pytest.mark.parametrize("dtype", DTYPES)
def test_spmm_column_equals_spmv(dtype):
    from gpu_util import run_spmv
    rng = np.random.default_rng(1)
    m, n, k = 4000, 500, 8
    A = gen.random_csr(m, n, rng.integers(0, 30, m), 2)
    B = rng.standard_normal((n, k)).astype(np.float32)
    Y, Y_ref, S = run_spmm(A, B.ravel(), k, None, 1.0, 0.0, dtype)
    assert_within(Y, Y_ref, S, dtype)


@pytest.mark.parametrize("name", ["c5k64", "c5k256"])
def test_workload_scaled(name):
    w = gen.workload(name, scale_down=3)
    for dtype in w.dtypes:
        Y, Y_ref, S = run_spmm(w.A, w.B, w.k, None, w.alpha, w.beta, dtype)
        assert_within(Y, Y_ref, S, dtype, what="%s %s" % (name, dtype))


@pytest.mark.parametrize("name", ["c5k64", "c5k256"])
def test_workload_full_size_sampled_rows(name):
    """Full size; the oracle computes 2048 sampled output rows (plus the first and last) one by one."""
    w = gen.workload(name)
    rng = np.random.default_rng(11)
    rows = np.unique(np.concatenate([[0, w.A.m - 1], rng.integers(0, w.A.m, 2048)])).astype(np.int64)
    for dtype in w.dtypes:
        Y, Y_ref, S = run_spmm(w.A, w.B, w.k, None, w.alpha, w.beta, dtype, rows=rows)
        assert_within(Y, Y_ref, S, dtype, what="%s %s full" % (name, dtype))


@pytest.mark.parametrize("dtype", DTYPES)
def test_host_buffer_entry_point(dtype):
    w = gen.workload("c5k64", scale_down=4)
    A = w.A
    vals, B = store(A.vals, dtype), store(w.B, dtype)
    Y = np.zeros(A.m * w.k, np.float32 if dtype == "f32" else np.uint16)
    b200sp.spmm_csr_host(A.m, A.n, A.nnz, w.k, A.row_ptr, A.col_idx, vals, B, Y, 1.0, 0.0, dtype)
    Y_ref, S = oracle.spmm_csr(A.m, A.n, w.k, A.row_ptr, A.col_idx, vals, B, None, 1.0, 0.0, dtype)
    assert_within(Y.reshape(A.m, w.k), Y_ref, S, dtype)


def test_output_larger_than_2_31_elements():
    """m * k > 2^31: the row-times-k offsets must be 64-bit.  BF16 storage, few columns (the kernel that holds a slice of B in
    shared memory) and the k-sliced kernel; only sampled rows are copied back and compared."""
    import torch
    from gpu_util import to_dev
    m, n, k = 600_000, 2048, 4096
    rng = np.random.default_rng(77)
    lens = rng.integers(4, 17, m)
    A = gen.random_csr(m, n, lens, seed=9, sort_cols=True)
    B = gen.to_bf16(rng.standard_normal(n * k).astype(np.float32))
    vals = gen.to_bf16(A.vals)
    d_rp, d_ci, d_va, d_B = to_dev(A.row_ptr), to_dev(A.col_idx), to_dev(vals), to_dev(B)
    rows = np.unique(np.concatenate([[0, m - 1, 524_288, 524_289], rng.integers(0, m, 300)])).astype(np.int64)
    Y_ref, S = oracle.spmm_csr(m, n, k, A.row_ptr, A.col_idx, vals, B, None, 1.0, 0.0, "bf16", rows=rows, nthreads=oracle.max_threads())
    for bstage in (1, 0):
        b200sp.b200sp_set_option("spmm_bstage", bstage)
        try:
            d_Y = torch.full((m * k,), 0x7FC0, dtype=torch.int16, device="cuda:0")      # NaN patterns: every entry must be overwritten
            b200sp.spmm_csr(m, n, A.nnz, k, d_rp, d_ci, d_va, d_B, d_Y, 1.0, 0.0, "bf16")
            torch.cuda.synchronize()
            Y = d_Y.view(m, k)[torch.from_numpy(rows).to("cuda:0")].cpu().numpy().view(np.uint16)
            assert_within(Y, Y_ref, S, "bf16", what="m*k > 2^31, bstage=%d" % bstage)
            del d_Y
        finally:
            b200sp.b200sp_set_option("spmm_bstage", 1)
            b200sp.b200sp_cache_clear()
    b200sp.b200sp_check()
