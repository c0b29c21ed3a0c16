"""GPU parity of the COO and ELL front ends (paper tasks 8, 9, 14, 15) against their CPU oracle."""
import numpy as np
import pytest
import torch

import gen
import oracle
import paper_2603_07169_b200 as b200sp
from gpu_util import assert_within, empty_out, store, to_dev, to_host

pytestmark = pytest.mark.gpu
DTYPES = ["f32", "bf16"]


def matrices():
    rng = np.random.default_rng(8)
    return {
        "power_law": gen.random_csr(6000, 900, (rng.pareto(1.3, 6000) * 3).astype(np.int64).clip(0, 3000), 1),
        "uniform16": gen.uniform_rows(5000, 5000, 16, 3),
        "stencil": gen.stencil27(12, 5),
        "short_ragged": gen.random_csr(4001, 333, rng.integers(0, 10, 4001), 2),
        "one_column": gen.random_csr(500, 1, rng.integers(0, 2, 500), 4, allow_dup=True),
        # rows of every size class of the CSC transpose plan: <= 32 (a thread sorts), 33-4096 (a CTA in shared memory), more (a CTA in global memory)
        "long_rows": gen.random_csr(700, 12000, np.concatenate([rng.integers(0, 40, 690), [33, 4096, 4097, 9000, 5000, 0, 64, 1, 100, 11000]]), 6),
    }


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("name", sorted(matrices()))
def test_coo_spmv_and_spmm(name, dtype):
    A = matrices()[name]
    rng = np.random.default_rng(1)
    r, c, v = gen.csr_to_coo(A)
    x = rng.standard_normal(A.n).astype(np.float32)
    y0 = rng.standard_normal(A.m).astype(np.float32)
    v_s, x_s, y0_s = store(v, dtype), store(x, dtype), store(y0, dtype)
    d_r, d_c, d_v, d_x = to_dev(r), to_dev(c), to_dev(v_s), to_dev(x_s)
    y = to_dev(y0_s).clone()
    b200sp.spmv_coo(A.m, A.n, A.nnz, d_r, d_c, d_v, d_x, y, 1.25, 0.5, dtype)
    torch.cuda.synchronize()
    y_ref, S = oracle.spmm_coo(A.m, A.n, 1, r, c, v_s, x_s, y0_s, 1.25, 0.5, dtype)
    y0f = y0 if dtype == "f32" else gen.bf16_to_f32(y0_s)
    assert_within(to_host(y, dtype), y_ref[:, 0], S[:, 0], dtype, 1.25, np.abs(0.5 * y0f.astype(np.float64)), what="coo spmv " + name)
    k = 24
    B = rng.standard_normal(A.n * k).astype(np.float32)
    B_s = store(B, dtype)
    Y = empty_out(A.m * k, dtype)
    b200sp.spmm_coo(A.m, A.n, A.nnz, k, d_r, d_c, d_v, to_dev(B_s), Y, 1.0, 0.0, dtype)
    torch.cuda.synchronize()
    Y_ref, S = oracle.spmm_coo(A.m, A.n, k, r, c, v_s, B_s, None, 1.0, 0.0, dtype)
    assert_within(to_host(Y, dtype).reshape(A.m, k), Y_ref, S, dtype, what="coo spmm " + name)
    b200sp.b200sp_cache_clear()


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("name", ["power_law", "uniform16", "stencil", "short_ragged", "long_rows", "one_column"])
def test_csc_spmv_and_spmm(name, dtype):
    A = matrices()[name]
    rng = np.random.default_rng(3)
    cp, ri, va = gen.csr_to_csc(A)
    x = rng.standard_normal(A.n).astype(np.float32)
    y0 = rng.standard_normal(A.m).astype(np.float32)
    v_s, x_s, y0_s = store(va, dtype), store(x, dtype), store(y0, dtype)
    d_cp, d_ri, d_v = to_dev(cp), to_dev(ri), to_dev(v_s)
    for rep in range(2):                                  # second call uses the cached transpose plan
        y = to_dev(y0_s).clone()
        b200sp.spmv_csc(A.m, A.n, A.nnz, d_cp, d_ri, d_v, to_dev(x_s), y, 0.5, -1.0, dtype)
        torch.cuda.synchronize()
        y_ref, S = oracle.spmm_csc(A.m, A.n, 1, cp, ri, v_s, x_s, y0_s, 0.5, -1.0, dtype)
        y0f = y0 if dtype == "f32" else gen.bf16_to_f32(y0_s)
        assert_within(to_host(y, dtype), y_ref[:, 0], S[:, 0], dtype, 1.0, np.abs(y0f.astype(np.float64)), what="csc spmv " + name)
    k = 16
    B = rng.standard_normal(A.n * k).astype(np.float32)
    B_s = store(B, dtype)
    Y = empty_out(A.m * k, dtype)
    b200sp.spmm_csc(A.m, A.n, A.nnz, k, d_cp, d_ri, d_v, to_dev(B_s), Y, 1.0, 0.0, dtype)
    torch.cuda.synchronize()
    Y_ref, S = oracle.spmm_csc(A.m, A.n, k, cp, ri, v_s, B_s, None, 1.0, 0.0, dtype)
    assert_within(to_host(Y, dtype).reshape(A.m, k), Y_ref, S, dtype, what="csc spmm " + name)
    b200sp.b200sp_cache_clear()


def test_csc_transpose_plan_is_built_on_the_device_and_reproducible():
    """The same CSC pattern planned twice (the cache dropped in between) gives bit-identical results: the order of a row's
    entries is fixed by their CSC positions, not by the order in which the placement kernel's atomics happened to run."""
    A = matrices()["long_rows"]
    cp, ri, va = gen.csr_to_csc(A)
    rng = np.random.default_rng(4)
    x = rng.standard_normal(A.n).astype(np.float32)
    d_cp, d_ri, d_v, d_x = to_dev(cp), to_dev(ri), to_dev(va), to_dev(x)
    outs = []
    for _ in range(3):
        y = empty_out(A.m, "f32")
        b200sp.spmv_csc(A.m, A.n, A.nnz, d_cp, d_ri, d_v, d_x, y, 1.0, 0.0, "f32")
        torch.cuda.synchronize()
        outs.append(y.cpu().numpy().copy())
        b200sp.b200sp_cache_drop(d_cp)
    assert np.array_equal(outs[0], outs[1]) and np.array_equal(outs[0], outs[2])
    # and equal, bit for bit, to the CSR path on the same matrix with columns in ascending order (the order the plan produces)
    order = np.lexsort((A.col_idx, np.repeat(np.arange(A.m), np.diff(A.row_ptr))))
    y = empty_out(A.m, "f32")
    b200sp.spmv_csr(A.m, A.n, A.nnz, to_dev(A.row_ptr), to_dev(A.col_idx[order]), to_dev(A.vals[order]), d_x, y, 1.0, 0.0, "f32")
    torch.cuda.synchronize()
    assert np.array_equal(outs[0], y.cpu().numpy())
    b200sp.b200sp_cache_clear()


def test_csc_inconsistent_pattern_is_refused():
    A = matrices()["short_ragged"]
    cp, ri, va = gen.csr_to_csc(A)
    bad = ri.copy(); bad[5] = A.m
    y = empty_out(A.m, "f32")
    with pytest.raises(b200sp.B200spError) as e:
        b200sp.spmv_csc(A.m, A.n, A.nnz, to_dev(cp), to_dev(bad), to_dev(va), to_dev(np.ones(A.n, np.float32)), y, 1.0, 0.0, "f32")
    assert e.value.status == 6
    b200sp.b200sp_cache_clear()


def test_coo_unsorted_rows_are_refused():
    A = matrices()["short_ragged"]
    r, c, v = gen.csr_to_coo(A)
    r = r.copy(); r[10], r[2000] = r[2000], r[10]
    t = [to_dev(a) for a in (r, c, v, np.ones(A.n, np.float32))]
    y = empty_out(A.m, "f32")
    with pytest.raises(b200sp.B200spError) as e:
        b200sp.spmv_coo(A.m, A.n, A.nnz, t[0], t[1], t[2], t[3], y, 1.0, 0.0, "f32")
    assert e.value.status == 2


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("name,extra", [("uniform16", 0), ("uniform16", 3), ("stencil", 0), ("stencil", 5), ("short_ragged", 0),
                                        ("short_ragged", 7), ("one_column", 0), ("power_law", 0)])
def test_ell_spmv_and_spmm(name, extra, dtype):
    A = matrices()[name]
    if name == "power_law":     # keep the padded matrix small: cap the longest rows
        A = gen.random_csr(A.m, A.n, np.minimum(np.diff(A.row_ptr), 200), 1)
    rng = np.random.default_rng(2)
    W, ci, va = gen.csr_to_ell(A, width=int(np.diff(A.row_ptr).max()) + extra, pad_value=77.0)
    x = rng.standard_normal(A.n).astype(np.float32)
    va_s, x_s = store(va, dtype), store(x, dtype)
    d_c, d_v = to_dev(ci), to_dev(va_s)
    y = empty_out(A.m, dtype)
    b200sp.spmv_ell(A.m, A.n, W, d_c, d_v, to_dev(x_s), y, 1.0, 0.0, dtype)
    torch.cuda.synchronize()
    y_ref, S = oracle.spmm_ell(A.m, A.n, W, 1, ci, va_s, x_s, None, 1.0, 0.0, dtype)
    assert_within(to_host(y, dtype), y_ref[:, 0], S[:, 0], dtype, what="ell spmv %s W=%d" % (name, W))
    for k in (32, 20):          # a multiple of the vector width and a ragged one
        B = rng.standard_normal(A.n * k).astype(np.float32)
        Y0 = rng.standard_normal(A.m * k).astype(np.float32)
        B_s, Y0_s = store(B, dtype), store(Y0, dtype)
        Y = to_dev(Y0_s).clone()
        b200sp.spmm_ell(A.m, A.n, W, k, d_c, d_v, to_dev(B_s), Y, -1.0, 2.0, dtype)
        torch.cuda.synchronize()
        Y_ref, S = oracle.spmm_ell(A.m, A.n, W, k, ci, va_s, B_s, Y0_s, -1.0, 2.0, dtype)
        y0f = Y0 if dtype == "f32" else gen.bf16_to_f32(Y0_s)
        assert_within(to_host(Y, dtype).reshape(A.m, k), Y_ref, S, dtype, 1.0, np.abs(2.0 * y0f.astype(np.float64)).reshape(A.m, k),
                      what="ell spmm %s k=%d" % (name, k))


def test_ell_all_padding_and_zero_width():
    m, n = 100, 10
    ci = np.full(m * 4, -1, np.int32)
    va = np.full(m * 4, np.nan, np.float32)          # padded values are never read into the sum
    y = empty_out(m, "f32")
    b200sp.spmv_ell(m, n, 4, to_dev(ci), to_dev(va), to_dev(np.ones(n, np.float32)), y, 1.0, 0.0, "f32")
    torch.cuda.synchronize()
    assert np.all(y.cpu().numpy() == 0)
    y0 = np.arange(m, dtype=np.float32)
    y = to_dev(y0).clone()
    b200sp.spmv_ell(m, n, 0, None, None, None, y, 1.0, 2.0, "f32")
    torch.cuda.synchronize()
    assert np.array_equal(y.cpu().numpy(), 2 * y0)
