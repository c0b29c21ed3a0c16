"""Failure paths of the library, reached without faulting, trapping or hanging the GPU:
 - a bounded wait in a kernel runs out (the producer is told to issue no copy, so nothing can be in flight), the kernel
   returns, b200sp_check reports B200SP_ERR_TIMEOUT once, and the next ordinary call is correct;
 - an allocation from the library's pool fails (injected on the host) in the plan pass and in the host-buffer entry points,
   the call returns B200SP_ERR_ALLOC and no device memory stays behind;
 - a plan is used with arguments that do not fit it; a cached plan is dropped by address."""
import numpy as np
import pytest
import torch

import gen
import oracle
import paper_2603_07169_b200 as b200sp
from gpu_util import assert_within, empty_out, run_spmm, run_spmv, store, to_dev, to_host

pytestmark = pytest.mark.gpu
TIMEOUT, ALLOC, INVALID = 7, 4, 1


def set_opts(**kw):
    for k, v in kw.items():
        b200sp.b200sp_set_option(k, v)


@pytest.mark.parametrize("which", ["row_direct", "ell_row_direct", "spmm_b_in_shared_memory"])
def test_bounded_wait_runs_out_and_the_library_recovers(which):
    rng = np.random.default_rng(3)
    b200sp.b200sp_check()                                   # start from a clear flag
    try:
        set_opts(spin_limit=1024, debug_no_copies=1)
        if which == "row_direct":
            b200sp.b200sp_set_option("spmv_kernel", 1)
            A = gen.stencil27(10, 2)
            d = [to_dev(a) for a in (A.row_ptr, A.col_idx, A.vals, np.ones(A.n, np.float32))]
            y = empty_out(A.m, "f32")
            b200sp.spmv_csr(A.m, A.n, A.nnz, d[0], d[1], d[2], d[3], y, 1.0, 0.0, "f32")
        elif which == "ell_row_direct":
            A = gen.stencil27(10, 2)
            W, ci, va = gen.csr_to_ell(A)
            assert W == 27                                   # an odd width: the staged kernel
            y = empty_out(A.m, "f32")
            b200sp.spmv_ell(A.m, A.n, W, to_dev(ci), to_dev(va), to_dev(np.ones(A.n, np.float32)), y, 1.0, 0.0, "f32")
        else:
            A = gen.random_csr(2000, 2048, rng.integers(20, 40, 2000), seed=5)
            k = 64
            d = [to_dev(a) for a in (A.row_ptr, A.col_idx, A.vals, rng.standard_normal(2048 * k).astype(np.float32))]
            Y = empty_out(A.m * k, "f32")
            b200sp.spmm_csr(A.m, A.n, A.nnz, k, d[0], d[1], d[2], d[3], Y, 1.0, 0.0, "f32")
        with pytest.raises(b200sp.B200spError) as e:        # the output of that launch is not looked at
            b200sp.b200sp_check()
        assert e.value.status == TIMEOUT
        b200sp.b200sp_check()                               # reported once: the flag is clear again
    finally:
        set_opts(spin_limit=1 << 20, debug_no_copies=0, spmv_kernel=-1)
        b200sp.b200sp_cache_clear()
    # the same problem through the same kernel, now with its copies: correct, and no flag
    if which == "spmm_b_in_shared_memory":
        B = rng.standard_normal(2048 * 64).astype(np.float32)
        Y, Y_ref, S = run_spmm(A, B, 64, None, 1.0, 0.0, "f32")
        assert_within(Y, Y_ref, S, "f32", what="after the timed-out SpMM")
    elif which == "ell_row_direct":
        x = rng.standard_normal(A.n).astype(np.float32)
        y = empty_out(A.m, "f32")
        b200sp.spmv_ell(A.m, A.n, W, to_dev(ci), to_dev(va), to_dev(x), y, 1.0, 0.0, "f32")
        torch.cuda.synchronize()
        y_ref, S = oracle.spmm_ell(A.m, A.n, W, 1, ci, va, x, None, 1.0, 0.0, "f32")
        assert_within(to_host(y, "f32"), y_ref[:, 0], S[:, 0], "f32", what="after the timed-out ELL SpMV")
    else:
        b200sp.b200sp_set_option("spmv_kernel", 1)
        try:
            x = rng.standard_normal(A.n).astype(np.float32)
            y, y_ref, S = run_spmv(A, x, None, 1.0, 0.0, "f32")
            assert_within(y, y_ref, S, "f32", what="after the timed-out SpMV")
        finally:
            b200sp.b200sp_set_option("spmv_kernel", -1)
    b200sp.b200sp_check()


def free_bytes():
    torch.cuda.synchronize()
    return torch.cuda.mem_get_info()[0]


def test_injected_allocation_failure_in_the_plan_pass_and_the_host_entry_points():
    w = gen.workload("c3", scale_down=3)
    A = w.A
    d_rp = to_dev(A.row_ptr)
    d_rest = [to_dev(a) for a in (A.col_idx, A.vals)]
    y0 = np.zeros(A.m, np.float32)
    # warm up: pools created, module loaded, one ordinary call of each kind
    plan = b200sp.b200sp_plan_create(A.m, A.n, A.nnz, d_rp)
    b200sp.b200sp_plan_destroy(plan)
    y = y0.copy()
    b200sp.spmv_csr_host(A.m, A.n, A.nnz, A.row_ptr, A.col_idx, A.vals, w.x, y, 1.0, 0.0, "f32")
    b200sp.spmv_csr_vec_host(A.m, A.n, A.nnz, d_rp, d_rest[0], d_rest[1], w.x, y, 1.0, 0.0, "f32")
    good = y.copy()
    b200sp.b200sp_cache_clear()
    base = free_bytes()

    def expect_alloc_error(nth, fn):
        b200sp.b200sp_set_option("fail_alloc_after", nth)
        try:
            with pytest.raises(b200sp.B200spError) as e:
                fn()
            assert e.value.status == ALLOC
        finally:
            b200sp.b200sp_set_option("fail_alloc_after", 0)
        b200sp.b200sp_cache_clear()
        assert abs(free_bytes() - base) <= (2 << 20), "device memory left behind after the failed call"

    expect_alloc_error(1, lambda: b200sp.b200sp_plan_create(A.m, A.n, A.nnz, d_rp))
    out = y0.copy()
    # host entry point: the first allocation is its staging block, the second the plan's block
    for nth in (1, 2):
        expect_alloc_error(nth, lambda: b200sp.spmv_csr_host(A.m, A.n, A.nnz, A.row_ptr, A.col_idx, A.vals, w.x, out, 1.0, 0.0, "f32"))
    # matrix-resident entry point: staging for x and y, then the cached plan of spmv_csr
    for nth in (1, 2):
        expect_alloc_error(nth, lambda: b200sp.spmv_csr_vec_host(A.m, A.n, A.nnz, d_rp, d_rest[0], d_rest[1], w.x, out, 1.0, 0.0, "f32"))
    # and everything still works afterwards
    b200sp.spmv_csr_host(A.m, A.n, A.nnz, A.row_ptr, A.col_idx, A.vals, w.x, out, 1.0, 0.0, "f32")
    assert np.array_equal(out, good)
    b200sp.b200sp_cache_clear()


def test_plan_used_with_arguments_that_do_not_fit_it():
    A = gen.random_csr(500, 300, np.full(500, 6), 3)
    d_rp, d_ci, d_va, d_x = to_dev(A.row_ptr), to_dev(A.col_idx), to_dev(A.vals), to_dev(np.ones(300, np.float32))
    y = empty_out(500, "f32")
    L = b200sp.lib()
    plan = b200sp.b200sp_plan_create(A.m, A.n, A.nnz, d_rp)
    try:
        n0 = b200sp.b200sp_launch_count()
        s = torch.cuda.current_stream().cuda_stream
        ptr = lambda t: t.data_ptr()
        assert L.b200sp_spmv(plan, ptr(d_ci), ptr(d_va), ptr(d_x), ptr(y), 1.0, 0.0, 5, s) == INVALID            # unknown dtype
        assert L.b200sp_spmv(plan, None, ptr(d_va), ptr(d_x), ptr(y), 1.0, 0.0, 0, s) == INVALID                  # missing col_idx
        assert L.b200sp_spmv(plan, ptr(d_ci), ptr(d_va), ptr(d_x), None, 1.0, 0.0, 0, s) == INVALID               # missing y
        assert L.b200sp_spmv(plan, ptr(d_ci) + 4, ptr(d_va), ptr(d_x), ptr(y), 1.0, 0.0, 0, s) == INVALID         # misaligned
        assert L.b200sp_spmm(plan, 0, ptr(d_ci), ptr(d_va), ptr(d_x), ptr(y), 1.0, 0.0, 0, s) == INVALID          # k = 0
        assert L.b200sp_spmm(plan, 1 << 31, ptr(d_ci), ptr(d_va), ptr(d_x), ptr(y), 1.0, 0.0, 0, s) == INVALID    # k too large
        assert b200sp.b200sp_launch_count() == n0                                                                 # nothing was launched
        # the binding refuses operands that are too short for the plan's sizes (BF16 storage where FP32 was planned for, a short y)
        with pytest.raises(b200sp.B200spError) as e:
            b200sp.b200sp_spmv(plan, d_ci, d_va, d_x, empty_out(100, "f32"), 1.0, 0.0, "f32")
        assert e.value.status == INVALID
        with pytest.raises(b200sp.B200spError) as e:
            b200sp.b200sp_spmv(plan, d_ci, d_va, d_x, y, 1.0, 0.0, "bf16")
        assert e.value.status == INVALID
        assert b200sp.b200sp_launch_count() == n0
        b200sp.b200sp_spmv(plan, d_ci, d_va, d_x, y, 1.0, 0.0, "f32")                                             # and the fitting call works
        torch.cuda.synchronize()
        y_ref, S = oracle.spmv_csr(A.m, A.n, A.row_ptr, A.col_idx, A.vals, np.ones(300, np.float32), None, 1.0, 0.0, "f32")
        assert_within(to_host(y, "f32"), y_ref, S, "f32")
    finally:
        b200sp.b200sp_plan_destroy(plan)


def test_cache_drop_forgets_one_pattern():
    """A cached plan is keyed on the address of row_ptr.  Rewriting that array in place without telling the library gives
    the stale plan (the documented hazard); b200sp_cache_drop(row_ptr) makes the next call plan again."""
    rng = np.random.default_rng(9)
    m, n = 3000, 5000
    A1 = gen.random_csr(m, n, np.full(m, 16), 1)                       # uniform rows: the kernel that never reads row_ptr
    lens = rng.integers(0, 31, m)
    lens[-1] += 16 * m - lens.sum()                                    # same nnz, other row structure (the last row takes the rest)
    assert 0 <= lens[-1] <= n
    A2 = gen.random_csr(m, n, lens, 2)
    assert A1.nnz == A2.nnz
    x = rng.standard_normal(n).astype(np.float32)
    d_rp, d_ci, d_va, d_x = to_dev(A1.row_ptr), to_dev(A1.col_idx), to_dev(A1.vals), to_dev(x)
    y = empty_out(m, "f32")
    b200sp.spmv_csr(m, n, A1.nnz, d_rp, d_ci, d_va, d_x, y, 1.0, 0.0, "f32")
    torch.cuda.synchronize()
    y_ref, S = oracle.spmv_csr(m, n, A1.row_ptr, A1.col_idx, A1.vals, x, None, 1.0, 0.0, "f32")
    assert_within(to_host(y, "f32"), y_ref, S, "f32")
    # the same device arrays now hold another matrix of the same sizes
    d_rp.copy_(torch.from_numpy(A2.row_ptr)); d_ci.copy_(torch.from_numpy(A2.col_idx)); d_va.copy_(torch.from_numpy(A2.vals))
    b200sp.b200sp_cache_drop(d_rp)
    b200sp.spmv_csr(m, n, A2.nnz, d_rp, d_ci, d_va, d_x, y, 1.0, 0.0, "f32")
    torch.cuda.synchronize()
    y_ref, S = oracle.spmv_csr(m, n, A2.row_ptr, A2.col_idx, A2.vals, x, None, 1.0, 0.0, "f32")
    assert_within(to_host(y, "f32"), y_ref, S, "f32", what="after b200sp_cache_drop")
    b200sp.b200sp_cache_drop(d_rp)
    b200sp.b200sp_cache_drop(d_x)                                      # unknown address: not an error
    b200sp.b200sp_cache_clear()


def test_host_entry_point_reuses_its_plan_and_forgets_it_on_request():
    w = gen.workload("c4", scale_down=2)
    A = w.A
    vals, x = store(A.vals, "bf16"), store(w.x, "bf16")
    y = np.zeros(A.m, np.uint16)
    b200sp.spmv_csr_host(A.m, A.n, A.nnz, A.row_ptr, A.col_idx, vals, x, y, 1.0, 0.0, "bf16")
    n0 = b200sp.b200sp_launch_count()
    y2 = np.zeros(A.m, np.uint16)
    b200sp.spmv_csr_host(A.m, A.n, A.nnz, A.row_ptr, A.col_idx, vals, x, y2, 1.0, 0.0, "bf16")
    assert b200sp.b200sp_checked_build() or b200sp.b200sp_launch_count() - n0 == 1            # the row-direct kernel alone: no plan pass, no column probe
    assert np.array_equal(y, y2)
    y_ref, S = oracle.spmv_csr(A.m, A.n, A.row_ptr, A.col_idx, vals, x, None, 1.0, 0.0, "bf16")
    assert_within(y2, y_ref, S, "bf16")
    b200sp.b200sp_cache_drop(A.row_ptr)
    n0 = b200sp.b200sp_launch_count()
    b200sp.spmv_csr_host(A.m, A.n, A.nnz, A.row_ptr, A.col_idx, vals, x, y2, 1.0, 0.0, "bf16")
    assert b200sp.b200sp_launch_count() - n0 > 1             # planned again
    assert np.array_equal(y, y2)
    b200sp.b200sp_cache_clear()


def test_pool_keep_mb_zero_returns_memory_at_every_synchronisation():
    """pool_keep_mb is read when a device's pool is created, so it is exercised in a process of its own."""
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    code = r'''
import numpy as np, torch, sys
sys.path.insert(0, %r)
import gen, paper_2603_07169_b200 as b
b.b200sp_set_option("pool_keep_mb", 0)
w = gen.workload("c2", scale_down=1); A = w.A
torch.cuda.init(); torch.zeros(1, device="cuda:0"); torch.cuda.synchronize()
y = w.y0.copy()
b.spmv_csr_host(A.m, A.n, A.nnz, A.row_ptr, A.col_idx, A.vals, w.x, y, w.alpha, w.beta, "f32")
b.b200sp_cache_clear()
f0 = torch.cuda.mem_get_info()[0]
ys = []
for _ in range(3):
    y = w.y0.copy()
    b.spmv_csr_host(A.m, A.n, A.nnz, A.row_ptr, A.col_idx, A.vals, w.x, y, w.alpha, w.beta, "f32")
    ys.append(y)
b.b200sp_cache_drop(A.row_ptr)
torch.cuda.synchronize()
f1 = torch.cuda.mem_get_info()[0]
assert all(np.array_equal(ys[0], v) for v in ys)
assert abs(f0 - f1) <= (4 << 20), (f0, f1)      # nothing is kept: 38 MB of staging went back at each synchronisation
print("ok")
''' % root
    out = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True, timeout=600)
    assert out.returncode == 0 and "ok" in out.stdout, out.stdout + out.stderr


def test_checked_build_refuses_an_inconsistent_matrix_before_touching_it():
    """libb200sp_check.so (built with -DB200SP_BOUNDS_CHECK) validates row_ptr and col_idx on the device before every compute
    call: a column index equal to n, or a decreasing row_ptr, comes back as B200SP_ERR_BAD_CSR with y untouched, and a
    consistent matrix gives the same result as the ordinary build.  It stands in for a memory checker: nothing traps.
    Run in a process of its own because the library file is chosen when the binding is imported."""
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    lib = os.path.join(root, "paper_2603_07169_b200", "libb200sp_check.so")
    if not os.path.exists(lib):
        from paper_2603_07169_b200 import build
        build.build(checked=True)
    code = r'''
import numpy as np, torch, sys
sys.path.insert(0, %r)
import gen, oracle, paper_2603_07169_b200 as b
assert b.b200sp_checked_build() == 1
dev = "cuda:0"
A = gen.random_csr(3000, 700, np.random.default_rng(1).integers(0, 30, 3000), 5)
x = np.random.default_rng(2).standard_normal(700).astype(np.float32)
up = lambda a: torch.from_numpy(a).to(dev)
d_rp, d_ci, d_va, d_x = up(A.row_ptr), up(A.col_idx), up(A.vals), up(x)
y = torch.full((A.m,), 7.0, device=dev)
b.spmv_csr(A.m, A.n, A.nnz, d_rp, d_ci, d_va, d_x, y, 1.0, 0.0, "f32")
torch.cuda.synchronize()
y_ref, S = oracle.spmv_csr(A.m, A.n, A.row_ptr, A.col_idx, A.vals, x, None, 1.0, 0.0, "f32")
assert oracle.tolerance_ratio(y.cpu().numpy(), y_ref, S, "f32")[0] <= 1.0
b.b200sp_cache_clear()
for what in ("col", "row"):
    ci, rp = A.col_idx.copy(), A.row_ptr.copy()
    if what == "col": ci[1234] = A.n
    else: rp[100] = rp[101] + 3
    y = torch.full((A.m,), 7.0, device=dev)
    n0 = b.b200sp_launch_count()
    try:
        b.spmv_csr(A.m, A.n, A.nnz, up(rp), up(ci), d_va, d_x, y, 1.0, 0.0, "f32")
        raise SystemExit("accepted a bad " + what)
    except b.B200spError as e:
        assert e.status == 6, e.status
    torch.cuda.synchronize()
    assert torch.all(y == 7.0)                     # no compute kernel ran
    b.b200sp_cache_clear()
Y = torch.full((A.m * 8,), 7.0, device=dev)
ci = A.col_idx.copy(); ci[5] = -1
try:
    b.spmm_csr(A.m, A.n, A.nnz, 8, d_rp, up(ci), d_va, up(np.ones(700 * 8, np.float32)), Y, 1.0, 0.0, "f32")
    raise SystemExit("accepted a negative column")
except b.B200spError as e:
    assert e.status == 6
assert torch.all(Y == 7.0)
print("ok")
''' % root
    env = dict(os.environ, B200SP_LIBRARY="libb200sp_check.so")
    out = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True, timeout=600, env=env)
    assert out.returncode == 0 and "ok" in out.stdout, out.stdout + out.stderr


def test_spmv_gather_probe_adds_every_product_and_refuses_bad_arguments():
    """The gather-phase probe on the caller's arrays: its per-thread partial sums add up to sum(vals * x[col_idx]) (FP32 and
    BF16 storage, with and without shared memory carved out), and out-of-range arguments launch nothing."""
    import torch
    import gen
    from gpu_util import to_dev
    rng = np.random.default_rng(4)
    A = gen.random_csr(3000, 5000, rng.integers(0, 60, 3000), seed=2)
    x = rng.standard_normal(A.n).astype(np.float32)
    nnz4 = A.nnz // 4 * 4
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    for dtype in ("f32", "bf16"):
        vals = A.vals if dtype == "f32" else gen.to_bf16(A.vals)
        xs = x if dtype == "f32" else gen.to_bf16(x)
        vf = A.vals if dtype == "f32" else gen.bf16_to_f32(vals)
        xf = x if dtype == "f32" else gen.bf16_to_f32(xs)
        want = float(np.dot(vf[:nnz4].astype(np.float64), xf[A.col_idx[:nnz4]].astype(np.float64)))
        scale = float(np.dot(np.abs(vf[:nnz4]).astype(np.float64), np.abs(xf[A.col_idx[:nnz4]]).astype(np.float64)))
        d_col, d_val, d_x = to_dev(A.col_idx), to_dev(vals), to_dev(xs)
        for kb in (0, 64):
            out = torch.zeros(sms * 1024, dtype=torch.float32, device="cuda:0")
            b200sp.b200sp_probe_spmv_gather(A.nnz, d_col, d_val, d_x, dtype, kb, out)
            torch.cuda.synchronize()
            got = float(out.double().sum())
            assert abs(got - want) <= 1e-5 * scale, (dtype, kb, got, want)
    out = torch.zeros(sms * 1024, dtype=torch.float32, device="cuda:0")
    for bad in (dict(nnz=2), dict(kb=201), dict(kb=-1)):
        with pytest.raises(b200sp.B200spError):
            b200sp.b200sp_probe_spmv_gather(bad.get("nnz", A.nnz), d_col, d_val, d_x, "f32", bad.get("kb", 0), out)
