"""Helpers for the GPU parity tests: upload a workload, call the C ABI through the binding, compare
with the CPU oracle under the acceptance bounds (FP32: 1e-5 * S + 1e-30; BF16: 8e-3 * |y_ref| + 1e-5 * S)."""
import numpy as np
import torch

import gen
import oracle
import paper_2603_07169_b200 as b200sp

DEV = "cuda:0"


def to_dev(a):
    """numpy array -> CUDA tensor (uint16 BF16 patterns travel as int16 bits)."""
    if a is None:
        return None
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).to(DEV)
    return torch.from_numpy(a).to(DEV)


def to_host(t, dtype):
    a = t.cpu().numpy()
    return a.view(np.uint16) if dtype == "bf16" else a


def store(a, dtype):
    """FP32 samples -> the stored array for this dtype (float32, or uint16 BF16 patterns)."""
    if a is None:
        return None
    return gen.to_bf16(a) if dtype == "bf16" else np.ascontiguousarray(a, np.float32)


def empty_out(count, dtype, fill_nan=True):
    t = torch.empty(count, dtype=torch.float32 if dtype == "f32" else torch.int16, device=DEV)
    if fill_nan:   # beta == 0 must ignore whatever is there, NaN included
        if dtype == "f32":
            t.fill_(float("nan"))
        else:
            t.fill_(0x7FC0)
    return t


def run_spmv(A, x, y0, alpha, beta, dtype, use_plan=False):
    """Returns (y as numpy in storage dtype, y_ref, S_ref)."""
    vals_s, x_s, y0_s = store(A.vals, dtype), store(x, dtype), store(y0, dtype)
    d_rp, d_ci, d_va, d_x = to_dev(A.row_ptr), to_dev(A.col_idx), to_dev(vals_s), to_dev(x_s)
    d_y = to_dev(y0_s).clone() if (beta != 0 and y0 is not None) else empty_out(A.m, dtype)
    if use_plan:
        plan = b200sp.b200sp_plan_create(A.m, A.n, A.nnz, d_rp)
        try:
            b200sp.b200sp_spmv(plan, d_ci, d_va, d_x, d_y, alpha, beta, dtype)
            torch.cuda.synchronize()
        finally:
            b200sp.b200sp_plan_destroy(plan)
    else:
        b200sp.spmv_csr(A.m, A.n, A.nnz, d_rp, d_ci, d_va, d_x, d_y, alpha, beta, dtype)
        torch.cuda.synchronize()
        b200sp.b200sp_cache_clear()
    y_ref, S_ref = oracle.spmv_csr(A.m, A.n, A.row_ptr, A.col_idx, vals_s, x_s, y0_s if beta != 0 else None, alpha, beta,
                                   dtype, nthreads=oracle.max_threads())
    return to_host(d_y, dtype), y_ref, S_ref


def run_spmm(A, B, k, Y0, alpha, beta, dtype, rows=None):
    vals_s, B_s, Y0_s = store(A.vals, dtype), store(B, dtype), store(Y0, dtype)
    d_rp, d_ci, d_va, d_B = to_dev(A.row_ptr), to_dev(A.col_idx), to_dev(vals_s), to_dev(B_s)
    d_Y = to_dev(Y0_s).clone() if (beta != 0 and Y0 is not None) else empty_out(A.m * k, dtype)
    b200sp.spmm_csr(A.m, A.n, A.nnz, k, d_rp, d_ci, d_va, d_B, d_Y, alpha, beta, dtype)
    torch.cuda.synchronize()
    b200sp.b200sp_cache_clear()
    Y_ref, S_ref = oracle.spmm_csr(A.m, A.n, k, A.row_ptr, A.col_idx, vals_s, B_s, Y0_s if beta != 0 else None, alpha, beta,
                                   dtype, rows=rows, nthreads=oracle.max_threads())
    Y = to_host(d_Y, dtype).reshape(A.m, k)
    if rows is not None:
        Y = Y[rows]
    return Y, Y_ref, S_ref


def assert_within(y, y_ref, S_ref, dtype, scale_S=1.0, extra=None, what=""):
    """The acceptance bound; scale_S and extra widen S for the labelled extension S' = |alpha| S + |beta y0|."""
    S = S_ref * scale_S + (extra if extra is not None else 0.0)
    ratio, idx = oracle.tolerance_ratio(y, y_ref, S, dtype)
    assert ratio <= 1.0, "%s: tolerance ratio %.3g at flat index %d (y_ref %r, S %r)" % (
        what, ratio, idx, y_ref.flat[idx], S.flat[idx])
    return ratio
