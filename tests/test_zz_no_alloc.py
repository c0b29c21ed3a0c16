"""spmv_csr_noalloc: the entry point for callers that may not allocate device memory (its scratch is a
fixed array inside the library).  Collected last on purpose: if it fails, a run that stops at the
first failure has already run everything else.  It is checked against the ordinary entry point
(spmv_csr) on two calls in a row that use different data, so stale scratch from the first call
would show in the second."""
import numpy as np
import pytest
import torch

import gen
import oracle
import paper_2603_07169_b200 as b200sp
from gpu_util import empty_out, store, to_dev, to_host

pytestmark = pytest.mark.gpu


def both_ways(A, x, y0, alpha, beta, dtype):
    """(y from spmv_csr_noalloc, y from spmv_csr, acceptance bound per row)."""
    vals_s, x_s, y0_s = store(A.vals, dtype), store(x, dtype), store(y0, dtype)
    d = [to_dev(a) for a in (A.row_ptr, A.col_idx, vals_s, x_s)]
    outs = []
    for fn in (b200sp.spmv_csr_noalloc, b200sp.spmv_csr):
        y = to_dev(y0_s).clone() if beta != 0 else empty_out(A.m, dtype)
        fn(A.m, A.n, A.nnz, d[0], d[1], d[2], d[3], y, alpha, beta, dtype)
        torch.cuda.synchronize()
        outs.append(to_host(y, dtype))
    b200sp.b200sp_cache_clear()
    y_ref, S = oracle.spmv_csr(A.m, A.n, A.row_ptr, A.col_idx, vals_s, x_s, y0_s if beta != 0 else None, alpha, beta, dtype,
                               nthreads=oracle.max_threads())
    S = abs(alpha) * S + (np.abs(beta * (y0_s if dtype == "f32" else gen.bf16_to_f32(y0_s)).astype(np.float64)) if beta != 0 else 0.0)
    bound = (1e-5 * S + 1e-30) if dtype == "f32" else (8e-3 * np.abs(y_ref) + 1e-5 * S)
    f = (lambda a: a.astype(np.float64)) if dtype == "f32" else (lambda a: gen.bf16_to_f32(a).astype(np.float64))
    return f(outs[0]), f(outs[1]), y_ref, bound


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_noalloc_matches_ordinary_entry_point_twice_in_a_row(dtype):
    rng = np.random.default_rng(5)
    # call 1: power-law rows (rows cut by tile boundaries exercise the carry / tail scratch)
    w = gen.workload("c3", scale_down=2)
    a, b, y_ref, bound = both_ways(w.A, w.x, None, 1.0, 0.0, dtype)
    assert np.all(np.abs(a - y_ref) <= bound) and np.all(np.abs(b - y_ref) <= bound)
    assert np.all(np.abs(a - b) <= 2 * bound)
    # call 2, straight after: a different, smaller matrix with other values, alpha and beta
    lens = rng.integers(0, 50, 30000)
    lens[100] = 20000
    A2 = gen.random_csr(30000, 5000, lens, 17)
    x2 = rng.standard_normal(5000).astype(np.float32)
    y02 = rng.standard_normal(30000).astype(np.float32)
    a, b, y_ref, bound = both_ways(A2, x2, y02, -0.5, 1.25, dtype)
    assert np.all(np.abs(a - y_ref) <= bound) and np.all(np.abs(b - y_ref) <= bound)
    assert np.all(np.abs(a - b) <= 2 * bound)


def test_noalloc_rejects_problems_beyond_its_scratch():
    lim = b200sp.b200sp_noalloc_max_items()
    assert lim == 65536 * 4096
    t = torch.zeros(64, dtype=torch.int32, device="cuda:0")
    n0 = b200sp.b200sp_launch_count()
    with pytest.raises(b200sp.B200spError) as e:
        # sizes only: nothing is launched or read when the limit is exceeded
        b200sp.spmv_csr_noalloc(lim // 2 + 1, 1000, lim // 2, t, t, t, t, t, 1.0, 0.0, "f32")
    assert e.value.status == 8
    assert b200sp.b200sp_launch_count() == n0


def test_noalloc_allocates_nothing_and_launches_only_its_three_kernels():
    """What the name promises: once the first call on the device has looked up the address of the built-in scratch, a call
    leaves the amount of free device memory exactly as it found it (no plan, no pool, no cache) and launches the split
    search, the merge-tile kernel and the carry fix-up, nothing else.  The sizes cover a problem whose rows + nonzeros are
    an exact multiple of the tile (4096), a row that spans more than three tiles, and a single-tile problem (no fix-up)."""
    rng = np.random.default_rng(17)
    lens = rng.integers(0, 9, 1000)
    lens[500] = 14000                                        # spans four tiles of 4096 merge items
    lens[-1] += (-(1000 + lens.sum())) % 4096                # rows + nonzeros = a multiple of 4096
    big = gen.random_csr(1000, 20000, lens, 3)
    assert (big.m + big.nnz) % 4096 == 0
    small = gen.random_csr(300, 100, rng.integers(0, 6, 300), 4)
    assert small.m + small.nnz <= 4096
    # every device buffer exists before the measured calls, so that the test's own allocations are not what is observed
    bufs = []
    for A in (big, small):
        x = rng.standard_normal(A.n).astype(np.float32)
        bufs.append((A, x, [to_dev(a) for a in (A.row_ptr, A.col_idx, A.vals, x)], empty_out(A.m, "f32")))
    A, x, d, y = bufs[0]
    b200sp.spmv_csr_noalloc(A.m, A.n, A.nnz, d[0], d[1], d[2], d[3], y, 1.0, 0.0, "f32")      # warm-up: module loaded, symbol looked up
    torch.cuda.synchronize()
    for (A, x, d, y), launches in zip(bufs, (3, 2)):
        unchanged = 0
        for _ in range(4):                                   # the second, third, ... call
            free0 = torch.cuda.mem_get_info()[0]
            n0 = b200sp.b200sp_launch_count()
            b200sp.spmv_csr_noalloc(A.m, A.n, A.nnz, d[0], d[1], d[2], d[3], y, 1.0, 0.0, "f32")
            torch.cuda.synchronize()
            unchanged += int(torch.cuda.mem_get_info()[0] == free0)
            assert b200sp.b200sp_checked_build() or b200sp.b200sp_launch_count() - n0 == launches
        # an allocation made by the call would show on every call; the driver's own housekeeping (a module loaded lazily on
        # the first launch of a kernel) may show once
        assert unchanged >= 3
        y_ref, S = oracle.spmv_csr(A.m, A.n, A.row_ptr, A.col_idx, A.vals, x, None, 1.0, 0.0, "f32")
        assert np.all(np.abs(to_host(y, "f32").astype(np.float64) - y_ref) <= 1e-5 * S + 1e-30)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_noalloc_two_calls_queued_back_to_back_on_one_stream(dtype):
    """Two calls with different matrices enqueued on the same stream with no synchronisation in between share the built-in
    scratch and are kept apart by stream order alone; both results must be right."""
    rng = np.random.default_rng(23)
    w = gen.workload("c3", scale_down=3)
    lens = rng.integers(0, 40, 20000)
    lens[7] = 30000
    A2 = gen.random_csr(20000, 40000, lens, 6)
    jobs = []
    for A, x in ((w.A, w.x), (A2, rng.standard_normal(A2.n).astype(np.float32))):
        vals_s, x_s = store(A.vals, dtype), store(x, dtype)
        jobs.append((A, vals_s, x_s, [to_dev(a) for a in (A.row_ptr, A.col_idx, vals_s, x_s)], empty_out(A.m, dtype)))
    torch.cuda.synchronize()
    for A, vals_s, x_s, d, y in jobs:                       # no synchronisation between the two calls
        b200sp.spmv_csr_noalloc(A.m, A.n, A.nnz, d[0], d[1], d[2], d[3], y, 1.0, 0.0, dtype)
    torch.cuda.synchronize()
    for A, vals_s, x_s, d, y in jobs:
        y_ref, S = oracle.spmv_csr(A.m, A.n, A.row_ptr, A.col_idx, vals_s, x_s, None, 1.0, 0.0, dtype, nthreads=oracle.max_threads())
        ratio, idx = oracle.tolerance_ratio(to_host(y, dtype), y_ref, S, dtype)
        assert ratio <= 1.0, (ratio, idx)
