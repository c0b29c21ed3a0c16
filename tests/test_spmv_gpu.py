"""GPU parity: CSR SpMV through the C ABI against the CPU oracle, element by element."""
import numpy as np
import pytest
import torch

import gen
import oracle
import paper_2603_07169_b200 as b200sp
from gpu_util import assert_within, empty_out, run_spmv, store, to_dev, to_host

pytestmark = pytest.mark.gpu

DTYPES = ["f32", "bf16"]


def ext_bound(A, S_ref, y0, alpha, beta):
    """Labelled extension of the bound for alpha != 1 / beta != 0: S' = |alpha| S + |beta y0|."""
    extra = np.abs(beta * y0.astype(np.float64)) if (beta != 0 and y0 is not None) else None
    return abs(alpha) if alpha != 0 else 1.0, extra


# ---------------------------------------------------------------- adversarial small shapes
def row_len_cases():
    rng = np.random.default_rng(0)
    cases = {
        "every_length_0_to_130": np.arange(131),
        "all_empty": np.zeros(1000, np.int64),
        "one_huge_row": np.array([3, 0, 100000, 5, 0, 0, 1]),
        "huge_first_and_last": np.array([20000, 1, 0, 2, 30000]),
        "single_row": np.array([9000]),
        "single_entry": np.array([1]),
        "many_empty_then_dense": np.concatenate([np.zeros(9000, np.int64), np.full(50, 700)]),
        "lengths_32_33": np.tile([32, 33], 700),
        "random_geometric": rng.geometric(0.08, 5000) - 1,
        "tile_exact": np.full(4096 // 17 * 3, 16),          # rows + nnz = multiple of the tile size
        "power_law": (rng.pareto(1.2, 3000) * 3).astype(np.int64).clip(0, 40000),
        "uniform_16": np.full(5003, 16),
        "uniform_27_ragged_rows": np.full(1001, 27),
        "uniform_64": np.full(777, 64),
        "uniform_4": np.full(4001, 4),
        "uniform_8": np.full(3001, 8),
        "uniform_32": np.full(1501, 32),
        "uniform_128": np.full(301, 128),
        "short_mixed_0_to_8": rng.integers(0, 9, 10007),
        "stencil_like": np.tile([8, 12, 18, 27, 27, 27, 27, 18], 500),
    }
    return cases


@pytest.fixture(params=[-1, 0, 1, 2, 3], ids=["auto", "merge_tile", "row_direct", "uniform", "subwarp"])
def kernel_choice(request):
    """Runs a test under each SpMV kernel selection (1 falls back to 0 inside the plan when rows are too long)."""
    b200sp.b200sp_set_option("spmv_kernel", request.param)
    yield request.param
    b200sp.b200sp_set_option("spmv_kernel", -1)
    b200sp.b200sp_check()


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("case", sorted(row_len_cases()))
def test_adversarial_row_lengths(case, dtype, kernel_choice):
    lens = row_len_cases()[case]
    m = len(lens)
    n = 777
    A = gen.random_csr(m, n, lens, seed=len(case), sort_cols=False, allow_dup=True)
    rng = np.random.default_rng(1)
    x = rng.standard_normal(n).astype(np.float32)
    y0 = rng.standard_normal(m).astype(np.float32)
    for alpha, beta in [(1.0, 0.0), (-1.25, 0.75)]:
        y, y_ref, S = run_spmv(A, x, y0, alpha, beta, dtype)
        sc, extra = ext_bound(A, S, store(y0, "f32") if dtype == "f32" else gen.bf16_to_f32(gen.to_bf16(y0)), alpha, beta)
        assert_within(y, y_ref, S, dtype, sc, extra, what="%s %s a=%g b=%g" % (case, dtype, alpha, beta))


@pytest.mark.parametrize("dtype", DTYPES)
def test_empty_rows_are_exactly_zero_and_nan_in_y_is_ignored(dtype):
    lens = np.array([0, 5, 0, 0, 40, 0])
    A = gen.random_csr(6, 50, lens, 5)
    x = np.ones(50, np.float32)
    y, y_ref, S = run_spmv(A, x, None, 1.0, 0.0, dtype)     # run_spmv pre-fills y with NaN
    yf = y if dtype == "f32" else gen.bf16_to_f32(y)
    assert np.all(np.isfinite(yf))
    assert yf[0] == 0 and yf[2] == 0 and yf[3] == 0 and yf[5] == 0
    assert_within(y, y_ref, S, dtype)


@pytest.mark.parametrize("dtype", DTYPES)
def test_n_equal_one_and_m_not_multiple_of_anything(dtype, kernel_choice):
    rng = np.random.default_rng(3)
    m = 4099
    lens = rng.integers(0, 4, m)
    A = gen.random_csr(m, 1, lens, 9)
    x = np.array([1.5], np.float32)
    y, y_ref, S = run_spmv(A, x, None, 1.0, 0.0, dtype)
    assert_within(y, y_ref, S, dtype)


@pytest.mark.parametrize("dtype", DTYPES)
def test_alpha_zero_and_no_nonzeros(dtype):
    m, n = 3000, 10
    A = gen.random_csr(m, n, np.full(m, 2), 1)
    rng = np.random.default_rng(0)
    y0 = rng.standard_normal(m).astype(np.float32)
    x = np.full(n, np.nan, np.float32)                        # alpha == 0: A and x are not read
    y, y_ref, S = run_spmv(A, np.ones(n, np.float32), y0, 0.0, 2.0, dtype)
    yf = y if dtype == "f32" else gen.bf16_to_f32(y)
    assert_within(y, y_ref, S, dtype, 1.0, np.abs(2.0 * y0.astype(np.float64)))
    Z = gen.random_csr(m, n, np.zeros(m, np.int64), 1)
    y, y_ref, S = run_spmv(Z, np.ones(n, np.float32), y0, 1.0, 0.0, dtype)
    yf = y if dtype == "f32" else gen.bf16_to_f32(y)
    assert np.all(yf == 0)
    y, y_ref, S = run_spmv(Z, np.ones(n, np.float32), y0, 1.0, -1.0, dtype)
    assert_within(y, y_ref, S, dtype, 1.0, np.abs(y0.astype(np.float64)))


def test_integer_data_is_exact_fp32():
    rng = np.random.default_rng(2)
    m, n = 20000, 300
    lens = rng.integers(0, 60, m)
    lens[17] = 9000
    A = gen.random_csr(m, n, lens, 4, integer_vals=True)
    x = rng.integers(-3, 4, n).astype(np.float32)
    y, y_ref, S = run_spmv(A, x, None, 1.0, 0.0, "f32")
    assert np.array_equal(y.astype(np.float64), y_ref)        # every partial sum is an exact integer


# ---------------------------------------------------------------- the measured workloads
@pytest.mark.parametrize("name,scale", [("c1", 0), ("c2", 2), ("c3", 2), ("c3p", 2), ("c4", 2)])
def test_workloads_scaled(name, scale, kernel_choice):
    w = gen.workload(name, scale_down=scale)
    for dtype in w.dtypes:
        y, y_ref, S = run_spmv(w.A, w.x, w.y0, w.alpha, w.beta, dtype, use_plan=(dtype == "bf16"))
        r = assert_within(y, y_ref, S, dtype, what="%s %s" % (name, dtype))   # the literal bound, S without alpha/beta
        assert r < 1.0


@pytest.mark.parametrize("name", ["c2", "c3", "c4"])
def test_workloads_full_size(name):
    """Full size in the launch configuration the benchmark times; the oracle runs on all host cores."""
    w = gen.workload(name)
    for dtype in w.dtypes:
        y, y_ref, S = run_spmv(w.A, w.x, w.y0, w.alpha, w.beta, dtype)
        assert_within(y, y_ref, S, dtype, what="%s %s full" % (name, dtype))


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("empty", [1, 0])
@pytest.mark.parametrize("items", [1024, 2048, 4096])
def test_merge_kernel_tile_sizes(items, empty, dtype):
    """The merge-tile kernel at its three tile sizes on power-law rows, every row length, and a long run of empty rows, with
    and without the list of non-empty rows."""
    b200sp.b200sp_set_option("spmv_kernel", 0)
    b200sp.b200sp_set_option("merge_items", items)
    b200sp.b200sp_set_option("merge_empty", empty)
    try:
        rng = np.random.default_rng(items)
        for name, lens in (("power_law", (rng.pareto(1.1, 40000) * 2).astype(np.int64).clip(0, 60000)),
                           ("every_length", np.arange(300)), ("empty_run", np.concatenate([np.zeros(20000, np.int64), [5000, 1, 0, 7]]))):
            A = gen.random_csr(len(lens), 3001, lens, seed=7)
            x = rng.standard_normal(3001).astype(np.float32)
            y0 = rng.standard_normal(len(lens)).astype(np.float32)
            y, y_ref, S = run_spmv(A, x, None, 1.0, 0.0, dtype)
            assert_within(y, y_ref, S, dtype, what="%s items=%d" % (name, items))
            y, y_ref, S = run_spmv(A, x, y0, 2.0, -0.5, dtype)
            y0f = y0 if dtype == "f32" else gen.bf16_to_f32(gen.to_bf16(y0))
            assert_within(y, y_ref, S, dtype, 2.0, np.abs(0.5 * y0f.astype(np.float64)), what="%s items=%d ab" % (name, items))
        b200sp.b200sp_check()
    finally:
        for k, v in (("spmv_kernel", -1), ("merge_items", 2048), ("merge_empty", 0)):
            b200sp.b200sp_set_option(k, v)


@pytest.mark.parametrize("kernel", [-1, 0, 3])
def test_positive_data_chains_stay_below_the_literal_fp32_bound(kernel):
    """All-positive data: rounding errors do not cancel, so this is the case closest to the bound 1e-5 * S.  No lane may add
    more than about 128 products in one chain, whichever kernel runs: one row of 4096 among rows of 3 (the sub-warp kernel
    must take its lane count from the longest row, not the mean), one row of 20,000, and 1,000 rows of 1,000."""
    rng = np.random.default_rng(8)
    b200sp.b200sp_set_option("spmv_kernel", kernel)
    try:
        for name, lens in (("4096_among_3", np.concatenate([np.full(3000, 3), [4096], np.full(3000, 3)])),
                           ("one_20000", np.concatenate([np.full(500, 5), [20000], np.full(500, 5)])),
                           ("rows_of_1000", np.full(1000, 1000))):
            n = 30000
            A = gen.random_csr(len(lens), n, lens, seed=len(name))
            A.vals[:] = rng.random(A.nnz).astype(np.float32) + 0.01
            x = rng.random(n).astype(np.float32) + 0.01
            y, y_ref, S = run_spmv(A, x, None, 1.0, 0.0, "f32")
            r = assert_within(y, y_ref, S, "f32", what="positive data %s kernel %d" % (name, kernel))
            assert r < 0.5, "%s kernel %d: ratio %.3g" % (name, kernel, r)
    finally:
        b200sp.b200sp_set_option("spmv_kernel", -1)


@pytest.mark.parametrize("dtype", DTYPES)
def test_naive_baseline_kernels(dtype):
    """The baselines of the speed-up metric are held to the same bound as the product kernels."""
    rng = np.random.default_rng(4)
    A = gen.paper_uniform(1500, 2048, 0.01, seed=3)
    x = rng.standard_normal(2048).astype(np.float32)
    vals_s, x_s = store(A.vals, dtype), store(x, dtype)
    d = [to_dev(a) for a in (A.row_ptr, A.col_idx, vals_s, x_s)]
    y = empty_out(A.m, dtype)
    b200sp.b200sp_spmv_naive(A.m, A.n, A.nnz, d[0], d[1], d[2], d[3], y, 1.0, 0.0, dtype)
    torch.cuda.synchronize()
    y_ref, S = oracle.spmv_csr(A.m, A.n, A.row_ptr, A.col_idx, vals_s, x_s, None, 1.0, 0.0, dtype)
    assert_within(to_host(y, dtype), y_ref, S, dtype, what="naive spmv")
    k = 24
    B = rng.standard_normal(2048 * k).astype(np.float32)
    B_s = store(B, dtype)
    Y = empty_out(A.m * k, dtype)
    b200sp.b200sp_spmm_naive(A.m, A.n, A.nnz, k, d[0], d[1], d[2], to_dev(B_s), Y, 1.0, 0.0, dtype)
    torch.cuda.synchronize()
    Y_ref, S = oracle.spmm_csr(A.m, A.n, k, A.row_ptr, A.col_idx, vals_s, B_s, None, 1.0, 0.0, dtype)
    assert_within(to_host(Y, dtype).reshape(A.m, k), Y_ref, S, dtype, what="naive spmm")


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("rows", [1024, 4096, 32768])
def test_paper_sized_spmv(rows, dtype):
    """The paper's own SpMV CSR sizes (Table 6, task 12): rows x 2048 at density 0.01."""
    A = gen.paper_uniform(rows, 2048, 0.01, seed=rows)
    assert A.nnz == int(rows * 2048 * 0.01)
    x = gen.uniform(2048, -1.0, 1.0, 5, 1)
    y, y_ref, S = run_spmv(A, x, None, 1.0, 0.0, dtype)
    assert_within(y, y_ref, S, dtype, what="paper rows=%d" % rows)


@pytest.mark.parametrize("dtype", DTYPES)
def test_short_rows_with_scattered_columns_take_the_merge_kernel(dtype):
    """Short irregular rows select the row-direct kernel from row_ptr alone; the column probe must send random columns to the
    merge-tile kernel (2 launches per call) and keep a banded matrix on the row-direct kernel (1 launch)."""
    rng = np.random.default_rng(12)
    m = 1 << 17                                       # > 2^20 nonzeros so that the small-problem kernel is not chosen
    lens = rng.poisson(12, m).clip(0, 40)
    A = gen.random_csr(m, m, lens, seed=4)            # uniform random columns
    x = rng.standard_normal(m).astype(np.float32)
    vals_s, x_s = store(A.vals, dtype), store(x, dtype)
    d = [to_dev(a) for a in (A.row_ptr, A.col_idx, vals_s, x_s)]
    y = empty_out(m, dtype)
    b200sp.spmv_csr(m, m, A.nnz, d[0], d[1], d[2], d[3], y, 1.0, 0.0, dtype)      # plan + probe
    n0 = b200sp.b200sp_launch_count()
    b200sp.spmv_csr(m, m, A.nnz, d[0], d[1], d[2], d[3], y, 1.0, 0.0, dtype)
    torch.cuda.synchronize()
    assert b200sp.b200sp_checked_build() or b200sp.b200sp_launch_count() - n0 == 2     # merge-tile kernel + carry fix-up
    y_ref, S = oracle.spmv_csr(m, m, A.row_ptr, A.col_idx, vals_s, x_s, None, 1.0, 0.0, dtype, nthreads=oracle.max_threads())
    assert_within(to_host(y, dtype), y_ref, S, dtype, what="scattered short rows")
    b200sp.b200sp_cache_clear()
    w = gen.workload("c4", scale_down=1)              # 80^3 stencil: banded
    B = w.A
    vals_s, x_s = store(B.vals, dtype), store(w.x, dtype)
    d = [to_dev(a) for a in (B.row_ptr, B.col_idx, vals_s, x_s)]
    y = empty_out(B.m, dtype)
    b200sp.spmv_csr(B.m, B.n, B.nnz, d[0], d[1], d[2], d[3], y, 1.0, 0.0, dtype)
    n0 = b200sp.b200sp_launch_count()
    b200sp.spmv_csr(B.m, B.n, B.nnz, d[0], d[1], d[2], d[3], y, 1.0, 0.0, dtype)
    torch.cuda.synchronize()
    assert b200sp.b200sp_checked_build() or b200sp.b200sp_launch_count() - n0 == 1     # row-direct kernel, no fix-up
    b200sp.b200sp_cache_clear()


# ---------------------------------------------------------------- determinism, plan, validation, host API
@pytest.mark.parametrize("dtype", DTYPES)
def test_bitwise_run_to_run_determinism(dtype):
    w = gen.workload("c3", scale_down=1)
    A = w.A
    d = [to_dev(a) for a in (A.row_ptr, A.col_idx, store(A.vals, dtype), store(w.x, dtype))]
    outs = []
    for _ in range(3):
        y = empty_out(A.m, dtype)
        b200sp.spmv_csr(A.m, A.n, A.nnz, d[0], d[1], d[2], d[3], y, 1.0, 0.0, dtype)
        torch.cuda.synchronize()
        outs.append(y.cpu().numpy().copy())
    b200sp.b200sp_cache_clear()
    assert np.array_equal(outs[0].view(np.uint8), outs[1].view(np.uint8))
    assert np.array_equal(outs[0].view(np.uint8), outs[2].view(np.uint8))


def test_plan_info_matches_numpy():
    w = gen.workload("c3", scale_down=2)
    A = w.A
    d_rp = to_dev(A.row_ptr)
    plan = b200sp.b200sp_plan_create(A.m, A.n, A.nnz, d_rp)
    info = b200sp.b200sp_plan_info(plan)
    b200sp.b200sp_plan_destroy(plan)
    L = np.diff(A.row_ptr).astype(np.int64)
    assert info["m"] == A.m and info["n"] == A.n and info["nnz"] == A.nnz
    assert info["min_row_len"] == L.min() and info["max_row_len"] == L.max()
    edges = [(0, 0), (1, 4), (5, 32), (33, 128), (129, 1024), (1025, 1 << 40)]
    for j, (lo, hi) in enumerate(edges):
        sel = (L >= lo) & (L <= hi)
        assert info["bin_rows"][j] == sel.sum() and info["bin_nnz"][j] == L[sel].sum()
    assert info["spmv_tile_items"] in (1024, 2048, 4096)
    assert info["spmv_tiles"] == -(-(A.m + A.nnz) // info["spmv_tile_items"])
    b200sp.b200sp_set_option("merge_empty", 1)      # the merge list over the non-empty rows only (61 % of this matrix's rows are empty)
    try:
        plan = b200sp.b200sp_plan_create(A.m, A.n, A.nnz, d_rp)
        info2 = b200sp.b200sp_plan_info(plan)
        b200sp.b200sp_plan_destroy(plan)
    finally:
        b200sp.b200sp_set_option("merge_empty", 0)
    assert info2["spmv_tiles"] == -(-(int((L > 0).sum()) + A.nnz) // info2["spmv_tile_items"])
    assert info["spmv_kernel"] == 0          # power-law rows: merge-tile kernel
    w = gen.workload("c4", scale_down=2)
    plan = b200sp.b200sp_plan_create(w.A.m, w.A.n, w.A.nnz, to_dev(w.A.row_ptr))
    info = b200sp.b200sp_plan_info(plan)
    b200sp.b200sp_plan_destroy(plan)
    assert info["spmv_kernel"] == 1 and info["max_row_len"] == 27      # short regular rows: row-direct kernel


def test_validate_csr():
    A = gen.random_csr(100, 40, np.full(100, 3), 1)
    d_rp, d_ci = to_dev(A.row_ptr), to_dev(A.col_idx)
    assert b200sp.b200sp_validate_csr(A.m, A.n, A.nnz, d_rp, d_ci) == 0
    bad = A.col_idx.copy(); bad[7] = 40
    assert b200sp.b200sp_validate_csr(A.m, A.n, A.nnz, d_rp, to_dev(bad)) == 6
    bad = A.row_ptr.copy(); bad[5] = bad[6] + 1
    assert b200sp.b200sp_validate_csr(A.m, A.n, A.nnz, to_dev(bad), d_ci) == 6
    bad = A.row_ptr.copy(); bad[-1] -= 1
    assert b200sp.b200sp_validate_csr(A.m, A.n, A.nnz, to_dev(bad), d_ci) == 6


@pytest.mark.parametrize("dtype", DTYPES)
def test_host_buffer_entry_point(dtype):
    w = gen.workload("c2", scale_down=3)
    A = w.A
    vals, x, y0 = store(A.vals, dtype), store(w.x, dtype), store(w.y0, dtype)
    y = y0.copy()
    b200sp.spmv_csr_host(A.m, A.n, A.nnz, A.row_ptr, A.col_idx, vals, x, y, w.alpha, w.beta, dtype)
    y_ref, S = oracle.spmv_csr(A.m, A.n, A.row_ptr, A.col_idx, vals, x, y0, w.alpha, w.beta, dtype)
    assert_within(y, y_ref, S, dtype)
    # matrix on the device, vectors on the host
    y2 = y0.copy()
    b200sp.spmv_csr_vec_host(A.m, A.n, A.nnz, to_dev(A.row_ptr), to_dev(A.col_idx), to_dev(vals), x, y2, w.alpha, w.beta, dtype)
    assert_within(y2, y_ref, S, dtype)
    b200sp.b200sp_cache_clear()


def test_library_pool_reuses_and_returns_memory():
    """Repeated host-buffer calls and plan builds draw from the library's own pool: device memory in use does not grow
    from call to call, results stay identical, and b200sp_cache_clear hands the pool's unused memory back."""
    import torch
    w = gen.workload("c2", scale_down=1)        # 2^18 rows, 4.2 M nonzeros: 38 MB of staging per call
    A = w.A
    y0 = w.y0.copy()
    b200sp.b200sp_cache_clear()
    torch.cuda.synchronize()
    free_start = torch.cuda.mem_get_info()[0]
    ys, frees = [], []
    for _ in range(6):
        y = y0.copy()
        b200sp.spmv_csr_host(A.m, A.n, A.nnz, A.row_ptr, A.col_idx, A.vals, w.x, y, w.alpha, w.beta, "f32")
        p = b200sp.b200sp_plan_create(A.m, A.n, A.nnz, to_dev(A.row_ptr))
        b200sp.b200sp_plan_destroy(p)
        ys.append(y)
        frees.append(torch.cuda.mem_get_info()[0])
    assert all(np.array_equal(ys[0], y) for y in ys[1:])
    assert max(frees[1:]) - min(frees[1:]) <= (8 << 20)          # steady after the first call
    assert free_start - frees[-1] >= (16 << 20)                  # the pool is holding the staging memory ...
    b200sp.b200sp_cache_clear()
    torch.cuda.empty_cache()
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] >= free_start - (8 << 20)    # ... and gives it back on request


@pytest.mark.parametrize("name,scale,dtype", [("c2", 2, "f32"), ("c2", 2, "bf16"), ("c3", 2, "f32"), ("c4", 2, "bf16"), ("c1", 0, "f32")])
def test_dependent_calls_back_to_back(name, scale, dtype):
    """Each call's input is the previous call's output, with no host synchronisation in between: the kernels are scheduled
    behind one another (programmatic stream serialisation) and must still see the previous result complete.  The chain has
    to be bit-identical to the same chain under plain stream order, and its first link has to match the oracle."""
    w = gen.workload(name, scale_down=scale)
    A = w.A
    assert A.m == A.n
    vals = store(A.vals, dtype)
    d_rp, d_ci, d_va = to_dev(A.row_ptr), to_dev(A.col_idx), to_dev(vals)
    x0 = store((w.x / 64.0).astype(np.float32), dtype)

    def chain(pdl, links):
        b200sp.b200sp_set_option("pdl", pdl)
        try:
            bufs = [to_dev(x0), empty_out(A.m, dtype)]
            for i in range(links):
                b200sp.spmv_csr(A.m, A.n, A.nnz, d_rp, d_ci, d_va, bufs[i % 2], bufs[(i + 1) % 2], 0.125, 0.0, dtype)
            torch.cuda.synchronize()
            return to_host(bufs[links % 2], dtype).copy()
        finally:
            b200sp.b200sp_set_option("pdl", 1)
            b200sp.b200sp_cache_clear()

    y1 = chain(1, 1)
    y_ref, S = oracle.spmv_csr(A.m, A.n, A.row_ptr, A.col_idx, vals, x0, None, 0.125, 0.0, dtype)
    assert_within(y1, y_ref, S, dtype, what="first link %s %s" % (name, dtype))
    for links in (2, 7):
        assert np.array_equal(chain(1, links), chain(0, links)), "chain of %d differs between launch modes" % links


def test_sizes_next_to_the_int32_limit():
    """nnz = 2^31 - 16, the largest the 32-bit CSR arrays allow with 16 nonzeros per row (m = 2^27 - 1): every product of an
    index and a size inside the kernels must be taken in 64 bits or stay below 2^31.  The matrix is made on the device (17 GB of
    col_idx and vals), the uniform-row, merge-tile and row-direct kernels each run it, and 4096 sampled rows plus the first and
    the last rows are compared with the oracle, which gets those rows as a small CSR matrix of their own."""
    dev = "cuda:0"
    if torch.cuda.mem_get_info()[0] < (40 << 30):
        pytest.skip("needs 40 GB of free device memory")
    m, n, per_row = (1 << 27) - 1, 1 << 20, 16
    nnz = m * per_row
    assert nnz == (1 << 31) - 16
    g = torch.Generator(device=dev); g.manual_seed(7)
    col = torch.randint(0, n, (nnz,), dtype=torch.int32, device=dev, generator=g)
    val = torch.empty(nnz, dtype=torch.float32, device=dev).normal_(generator=g)
    row_ptr = (torch.arange(m + 1, dtype=torch.int64, device=dev) * per_row).to(torch.int32)
    assert int(row_ptr[-1]) == nnz
    x_h = np.random.default_rng(3).standard_normal(n).astype(np.float32)
    x = torch.from_numpy(x_h).to(dev)
    rows = np.unique(np.concatenate([np.arange(0, 64), np.arange(m - 64, m), np.random.default_rng(4).integers(0, m, 4096)])).astype(np.int64)
    idx = (torch.from_numpy(rows).to(dev)[:, None] * per_row + torch.arange(per_row, device=dev)[None, :]).reshape(-1)
    sub_col = col[idx].cpu().numpy()
    sub_val = val[idx].cpu().numpy()
    sub_rp = (np.arange(len(rows) + 1) * per_row).astype(np.int32)
    y_ref, S = oracle.spmv_csr(len(rows), n, sub_rp, sub_col, sub_val, x_h, None, 1.0, 0.0, "f32")
    d_rows = torch.from_numpy(rows).to(dev)
    try:
        for kernel in (2, 0, 1):
            b200sp.b200sp_set_option("spmv_kernel", kernel)
            y = torch.full((m,), float("nan"), dtype=torch.float32, device=dev)
            b200sp.spmv_csr(m, n, nnz, row_ptr, col, val, x, y, 1.0, 0.0, "f32")
            torch.cuda.synchronize()
            assert not bool(torch.isnan(y).any()), "kernel %d left rows unwritten" % kernel
            assert_within(y[d_rows].cpu().numpy(), y_ref, S, "f32", what="nnz = 2^31 - 16, kernel %d" % kernel)
            b200sp.b200sp_cache_clear()
            del y
        b200sp.b200sp_check()
    finally:
        b200sp.b200sp_set_option("spmv_kernel", -1)
        b200sp.b200sp_cache_clear()
        del col, val, row_ptr
        torch.cuda.empty_cache()


def test_plan_log_line(capfd):
    """With the switch "log" (B200SP_LOG=1 in the environment) every plan that is built reports its row statistics and the kernel chosen."""
    w = gen.workload("c3", scale_down=3)
    A = w.A
    b200sp.b200sp_set_option("log", 1)
    try:
        plan = b200sp.b200sp_plan_create(A.m, A.n, A.nnz, to_dev(A.row_ptr))
        b200sp.b200sp_plan_destroy(plan)
    finally:
        b200sp.b200sp_set_option("log", 0)
    err = capfd.readouterr().err
    L = np.diff(A.row_ptr)
    assert "b200sp plan: m=%d n=%d nnz=%d" % (A.m, A.n, A.nnz) in err, err
    assert "max=%d" % L.max() in err and "= %d|" % int((L == 0).sum()) in err, err
    assert any("spmv kernel=" + k in err for k in ("merge-tile", "row-direct", "uniform-row", "sub-warp")), err
