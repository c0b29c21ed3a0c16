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
    with pytest.raises(b200sp.B200spError) as e:
        # sizes only: nothing is launched or read when the limit is exceeded
        b200sp.spmv_csr_noalloc(lim // 2 + 1, 1000, lim // 2, t, t, t, t, t, 1.0, 0.0, "f32")
    assert e.value.status == 8
