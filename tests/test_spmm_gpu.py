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


@pytest.mark.parametrize("sliced", [1, 0])
@pytest.mark.parametrize("k", [3, 17, 64, 256])
def test_positive_data_chains_stay_below_the_literal_fp32_bound(k, sliced):
    """All-positive data, where rounding errors do not cancel.  No lane adds more than about 128 products in one chain:
    rows of up to 128 nonzeros are added in sequence, rows of 129-1024 in blocks of 128 whose sums form a second chain,
    longer rows by a CTA with blocks of 64 and a pairwise tree.  Rows of 128, 129, 1024, 1025 and 20,000 nonzeros, with k a
    multiple of the vector width and not (k = 3, 17: scalar lanes)."""
    rng = np.random.default_rng(5)
    lens = np.concatenate([np.full(100, 128), np.full(100, 129), np.full(60, 1024), np.full(10, 1025), [20000], np.full(50, 7)])
    n = 30000
    b200sp.b200sp_set_option("spmm_sliced", sliced)
    try:
        A = gen.random_csr(len(lens), n, lens, seed=1024)
        A.vals[:] = rng.random(A.nnz).astype(np.float32) + 0.01
        B = rng.random(n * k).astype(np.float32) + 0.01
        Y, Y_ref, S = run_spmm(A, B, k, None, 1.0, 0.0, "f32")
        r = assert_within(Y, Y_ref, S, "f32", what="positive data k=%d sliced=%d" % (k, sliced))
        assert r < 0.5, "k=%d sliced=%d: ratio %.3g" % (k, sliced, r)
    finally:
        b200sp.b200sp_set_option("spmm_sliced", 1)


def test_positive_data_few_columns_kernel():
    """The kernel that holds a slice of B in shared memory, rows of up to 2048 positive products (duplicates allowed)."""
    rng = np.random.default_rng(6)
    lens = np.concatenate([np.full(50, 2048), np.full(50, 1500), np.full(2000, 20), [6000]])
    A = gen.random_csr(len(lens), 2048, lens, seed=3, allow_dup=True)
    A.vals[:] = rng.random(A.nnz).astype(np.float32) + 0.01
    B = rng.random(2048 * 64).astype(np.float32) + 0.01
    Y, Y_ref, S = run_spmm(A, B, 64, None, 1.0, 0.0, "f32")
    assert assert_within(Y, Y_ref, S, "f32", what="positive data, B in shared memory") < 0.5


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


@pytest.mark.parametrize("name", ["c5k64", "c5k256", "c3k64"])
def test_workload_scaled(name):
    w = gen.workload(name, scale_down=3)
    for dtype in w.dtypes:
        Y, Y_ref, S = run_spmm(w.A, w.B, w.k, None, w.alpha, w.beta, dtype)
        assert_within(Y, Y_ref, S, dtype, what="%s %s" % (name, dtype))


def test_workload_full_size_every_entry_k64():
    """c5 with k = 64 at full size, both dtypes: every one of the 33.5 M output entries against the oracle."""
    w = gen.workload("c5k64")
    for dtype in w.dtypes:
        Y, Y_ref, S = run_spmm(w.A, w.B, w.k, None, w.alpha, w.beta, dtype)
        assert_within(Y, Y_ref, S, dtype, what="c5k64 %s full, all rows" % dtype)
        del Y, Y_ref, S


def test_power_law_spmm_full_size_sampled_rows():
    """The R-MAT matrix of the power-law workload times a dense n x 64 B at full size (the nnz-balanced kernel): 8192 sampled
    rows plus the 64 longest rows, the first and the last row, and a run of rows around the longest one."""
    w = gen.workload("c3k64")
    L = np.diff(w.A.row_ptr)
    rng = np.random.default_rng(13)
    longest = np.argsort(L)[-64:]
    rows = np.unique(np.concatenate([[0, w.A.m - 1], longest, np.arange(max(0, longest[-1] - 8), min(w.A.m, longest[-1] + 8)),
                                     rng.integers(0, w.A.m, 8192)])).astype(np.int64)
    for dtype in w.dtypes:
        Y, Y_ref, S = run_spmm(w.A, w.B, w.k, None, w.alpha, w.beta, dtype, rows=rows)
        assert_within(Y, Y_ref, S, dtype, what="c3k64 %s full" % dtype)


def test_workload_full_size_sampled_rows_k256():
    """c5 with k = 256 at full size; the oracle computes 8192 sampled output rows (plus the first and last of every block of
    2^16 rows) one by one."""
    w = gen.workload("c5k256")
    rng = np.random.default_rng(11)
    edges = np.arange(0, w.A.m + 1, 1 << 16)
    rows = np.unique(np.concatenate([edges[:-1], edges[1:] - 1, rng.integers(0, w.A.m, 8192)])).astype(np.int64)
    for dtype in w.dtypes:
        Y, Y_ref, S = run_spmm(w.A, w.B, w.k, None, w.alpha, w.beta, dtype, rows=rows)
        assert_within(Y, Y_ref, S, dtype, what="c5k256 %s full" % dtype)


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


def flat_row_cases():
    rng = np.random.default_rng(0)
    return {
        "every_length_0_to_130": np.arange(131),
        "all_empty_but_one": np.concatenate([np.zeros(3000, np.int64), [5], np.zeros(3000, np.int64)]),
        "one_huge_row": np.array([3, 0, 100000, 5, 0, 0, 1]),
        "huge_first_and_last": np.array([20000, 1, 0, 2, 30000]),
        "single_row": np.array([9000]),
        "single_entry": np.array([1]),
        "rows_of_32": np.full(700, 32),                      # chunks and rows coincide
        "rows_of_31_33": np.tile([31, 33], 400),             # every chunk boundary cuts a row
        "tile_exact": np.full(64, 1024),                     # rows and tiles coincide
        "power_law": (rng.pareto(1.2, 3000) * 3).astype(np.int64).clip(0, 40000),
        "long_run_of_empty_rows_inside_a_tile": np.concatenate([[7], np.zeros(5000, np.int64), [9], np.zeros(2000, np.int64), [2000]]),
    }


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("case", sorted(flat_row_cases()))
def test_nnz_balanced_kernel_adversarial_rows(case, dtype):
    """The nnz-balanced SpMM kernel (a chunk of 32 nonzeros per lane group, carries between chunks and tiles) forced on row-length
    patterns that hit every branch: rows inside a chunk, rows cut by chunk and by tile boundaries, rows spanning many tiles,
    runs of empty rows longer than the tile's staged row bounds, k that is and is not a multiple of a slice, beta != 0."""
    lens = flat_row_cases()[case]
    m, n = len(lens), 777
    A = gen.random_csr(m, n, lens, seed=len(case), sort_cols=False, allow_dup=True)
    rng = np.random.default_rng(2)
    b200sp.b200sp_set_option("spmm_flat", 1)
    b200sp.b200sp_set_option("spmm_bstage", 0)
    try:
        for k in (64, 72):
            B = rng.standard_normal(n * k).astype(np.float32)
            Y0 = rng.standard_normal(m * k).astype(np.float32)
            Y, Y_ref, S = run_spmm(A, B, k, None, 1.0, 0.0, dtype)
            assert_within(Y, Y_ref, S, dtype, what="flat %s k=%d" % (case, k))
            Y, Y_ref, S = run_spmm(A, B, k, Y0, -0.5, 1.25, dtype)
            y0f = Y0 if dtype == "f32" else gen.bf16_to_f32(gen.to_bf16(Y0))
            assert_within(Y, Y_ref, S, dtype, 1.0, np.abs(1.25 * y0f.astype(np.float64)).reshape(m, k), what="flat %s k=%d ab" % (case, k))
    finally:
        b200sp.b200sp_set_option("spmm_flat", 2)
        b200sp.b200sp_set_option("spmm_bstage", 1)


def test_nnz_balanced_kernel_is_reproducible_and_keeps_chains_short():
    """Bit-identical results from run to run (the carries are added in a fixed order), and all-positive data on rows of up to
    60,000 nonzeros stays far below the literal FP32 bound."""
    import torch
    from gpu_util import empty_out, store, to_dev
    rng = np.random.default_rng(9)
    lens = (rng.pareto(1.1, 20000) * 2).astype(np.int64).clip(0, 60000)
    n, k = 50000, 64
    A = gen.random_csr(len(lens), n, lens, seed=4)
    A.vals[:] = rng.random(A.nnz).astype(np.float32) + 0.01
    B = rng.random(n * k).astype(np.float32) + 0.01
    b200sp.b200sp_set_option("spmm_flat", 1)
    try:
        Y, Y_ref, S = run_spmm(A, B, k, None, 1.0, 0.0, "f32")
        assert assert_within(Y, Y_ref, S, "f32", what="flat, positive data") < 0.5
        d = [to_dev(a) for a in (A.row_ptr, A.col_idx, A.vals, B)]
        outs = []
        for _ in range(3):
            Yd = empty_out(A.m * k, "f32")
            b200sp.spmm_csr(A.m, A.n, A.nnz, k, d[0], d[1], d[2], d[3], Yd, 1.0, 0.0, "f32")
            torch.cuda.synchronize()
            outs.append(Yd.cpu().numpy().copy())
        assert np.array_equal(outs[0], outs[1]) and np.array_equal(outs[0], outs[2])
        assert np.array_equal(outs[0].reshape(A.m, k), Y)
    finally:
        b200sp.b200sp_set_option("spmm_flat", 2)
        b200sp.b200sp_cache_clear()


def quad_row_cases():
    rng = np.random.default_rng(1)
    return {
        "every_length_0_to_70": np.tile(np.arange(71), 3),           # every remainder modulo four, lengths changing inside blocks
        "all_empty_but_few": np.concatenate([np.zeros(500, np.int64), [5000], np.zeros(500, np.int64), [3, 1024, 1025]]),
        "rows_at_the_long_row_limit": np.array([1023, 1024, 1025, 1026, 4096, 0, 1, 2, 3, 4, 5000, 1024, 1024]),
        "only_long_rows": np.array([3000, 2000, 1500]),
        "single_row": np.array([4000]),
        "one_block_less_one": np.full(7, 24),
        "one_block_plus_one": np.full(17, 24),
        "equal_rows": np.full(4096, 20),
        "binomial": rng.binomial(2048, 0.01, 5000),
        "more_quads_than_a_warp_buffer": np.concatenate([np.full(40, 900), np.full(900, 40)]),
    }


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("n", [120, 2048, 5000])
@pytest.mark.parametrize("case", sorted(quad_row_cases()))
def test_b_in_shared_memory_sorted_quads_adversarial_rows(case, n, dtype):
    """The kernel that holds a slice of B in shared memory, on its re-laid copy of A (rows sorted by length into blocks, quads
    interleaved, entries ordered by bank class): all three slice widths (8, 4, 2 lanes per row: n = 120, 2048, 5000), every
    row-length remainder, list lengths around a block, rows on both sides of the long-row limit, blocks larger than a warp's
    buffer (read from global memory), k that is and is not a multiple of the slice, beta != 0."""
    lens = quad_row_cases()[case]
    m = len(lens)
    if lens.sum() < 4 * n:                        # the kernel is chosen when nnz >= 4 n
        lens = np.concatenate([lens, np.full((4 * n - lens.sum()) // 16 + 1, 16)])
        m = len(lens)
    A = gen.random_csr(m, n, lens, seed=len(case) + n, sort_cols=False, allow_dup=True)
    rng = np.random.default_rng(3)
    for k in (64, 72):
        B = rng.standard_normal(n * k).astype(np.float32)
        Y0 = rng.standard_normal(m * k).astype(np.float32)
        Y, Y_ref, S = run_spmm(A, B, k, None, 1.0, 0.0, dtype)
        assert_within(Y, Y_ref, S, dtype, what="quads %s n=%d k=%d" % (case, n, k))
        Y, Y_ref, S = run_spmm(A, B, k, Y0, -0.5, 1.25, dtype)
        y0f = Y0 if dtype == "f32" else gen.bf16_to_f32(gen.to_bf16(Y0))
        assert_within(Y, Y_ref, S, dtype, 1.0, np.abs(1.25 * y0f.astype(np.float64)).reshape(m, k), what="quads %s n=%d k=%d ab" % (case, n, k))
    b200sp.b200sp_check()


def test_b_in_shared_memory_sorted_quads_reproducible_exact_and_nonfinite():
    """Small-integer data: every product and sum is exact, so the result equals the oracle's bit for bit whatever the order of a
    row's products; three runs agree bit for bit; a row whose padded last quad sits next to an infinite entry of B stays
    infinite (padding is never multiplied); the plan's sorted order is reused by a second call with other values."""
    import torch
    from gpu_util import empty_out, to_dev
    rng = np.random.default_rng(12)
    n, k = 2048, 128
    lens = rng.binomial(2048, 0.01, 3000)
    lens[5] = 1                                   # one entry: three padded slots in its only quad
    A = gen.random_csr(len(lens), n, lens, seed=8, integer_vals=True)
    B = rng.integers(-3, 4, n * k).astype(np.float32)
    Y, Y_ref, S = run_spmm(A, B, k, None, 1.0, 0.0, "f32")
    assert np.array_equal(Y.astype(np.float64), Y_ref)
    d = [to_dev(a) for a in (A.row_ptr, A.col_idx, A.vals, B)]
    outs = []
    for _ in range(3):
        Yd = empty_out(A.m * k, "f32")
        b200sp.spmm_csr(A.m, A.n, A.nnz, k, d[0], d[1], d[2], d[3], Yd, 1.0, 0.0, "f32")
        torch.cuda.synchronize()
        outs.append(Yd.cpu().numpy().copy())
    assert np.array_equal(outs[0], outs[1]) and np.array_equal(outs[0], outs[2])
    assert np.array_equal(outs[0].reshape(A.m, k), Y)
    # offset 0 (the padding's) is row 0 of B: make it infinite; row 5 (one entry, another column) must not see it
    c5 = int(A.col_idx[A.row_ptr[5]])
    if c5 == 0:
        A.col_idx[A.row_ptr[5]] = c5 = 7
    B2 = B.copy()
    B2[:k] = np.inf
    A.vals[A.row_ptr[5]] = 2.0
    Y2, Y2_ref, _ = run_spmm(A, B2, k, None, 1.0, 0.0, "f32")
    assert np.all(np.isfinite(Y2[5])) and np.array_equal(Y2[5].astype(np.float64), Y2_ref[5])
    rows_with_col0 = np.unique(np.repeat(np.arange(A.m), np.diff(A.row_ptr))[A.col_idx == 0])
    assert len(rows_with_col0) > 0 and not np.any(np.isfinite(Y2[rows_with_col0]))
    b200sp.b200sp_check()
