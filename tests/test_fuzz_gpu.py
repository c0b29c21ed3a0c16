"""Randomised parity: many small and medium matrices with random shapes, row-length laws, column laws, scalars and dtypes
through every SpMV / SpMM front end, each checked element by element against the CPU oracle."""
import numpy as np
import pytest
import torch

import gen
import oracle
import paper_2603_07169_b200 as b200sp
from gpu_util import assert_within, run_spmm, run_spmv

pytestmark = pytest.mark.gpu


def random_matrix(rng, case):
    m = int(rng.choice([1, 2, 31, 257, 1000, 4099, 20000, 70001]))
    n = int(rng.choice([1, 7, 64, 1000, 30011]))
    law = case % 6
    if law == 0:
        lens = rng.integers(0, 9, m)
    elif law == 1:
        lens = np.full(m, int(rng.choice([4, 8, 12, 16, 27, 32, 64])))
    elif law == 2:
        lens = (rng.pareto(1.1, m) * 2).astype(np.int64).clip(0, 30000)
    elif law == 3:
        lens = rng.poisson(20, m)
    elif law == 4:
        lens = np.where(rng.random(m) < 0.9, 0, rng.integers(1, 300, m))
    else:
        lens = rng.geometric(0.2, m) - 1
        lens[rng.integers(0, m)] = 9000
    lens = np.minimum(lens, 40000)
    if lens.sum() > 3_000_000:
        lens = (lens * (3_000_000 / lens.sum())).astype(np.int64)
    A = gen.random_csr(m, n, lens, seed=case, sort_cols=bool(case & 1), allow_dup=True)
    if case % 3 == 0 and n > 64:       # banded columns: exercises the column-locality probe's "local" verdict
        rows = np.repeat(np.arange(m), np.diff(A.row_ptr))
        A.col_idx[:] = np.clip((rows * n) // max(m, 1) + rng.integers(-8, 9, A.nnz), 0, n - 1).astype(np.int32)
    return A


@pytest.mark.parametrize("case", range(36))
def test_spmv_fuzz(case):
    rng = np.random.default_rng(1000 + case)
    A = random_matrix(rng, case)
    dtype = "bf16" if case % 2 else "f32"
    alpha, beta = [(1.0, 0.0), (-0.5, 1.5), (2.0, -1.0), (0.0, 0.5)][case % 4]
    x = rng.standard_normal(A.n).astype(np.float32)
    y0 = rng.standard_normal(A.m).astype(np.float32)
    y, y_ref, S = run_spmv(A, x, y0, alpha, beta, dtype, use_plan=bool(case % 5 == 0))
    y0f = y0 if dtype == "f32" else gen.bf16_to_f32(gen.to_bf16(y0))
    assert_within(y, y_ref, S, dtype, max(abs(alpha), 1.0), np.abs(beta * y0f.astype(np.float64)), what="fuzz spmv case %d" % case)
    b200sp.b200sp_check()


@pytest.mark.parametrize("case", range(18))
def test_spmm_fuzz(case):
    rng = np.random.default_rng(2000 + case)
    A = random_matrix(rng, case + 1)
    if A.nnz > 400_000:
        pytest.skip("kept small for the oracle")
    k = int(rng.choice([1, 4, 8, 24, 33, 64, 96, 136]))
    dtype = "bf16" if case % 2 else "f32"
    alpha, beta = [(1.0, 0.0), (1.5, -0.5), (-1.0, 1.0)][case % 3]
    B = rng.standard_normal(A.n * k).astype(np.float32)
    Y0 = rng.standard_normal(A.m * k).astype(np.float32)
    Y, Y_ref, S = run_spmm(A, B, k, Y0, alpha, beta, dtype)
    y0f = Y0 if dtype == "f32" else gen.bf16_to_f32(gen.to_bf16(Y0))
    assert_within(Y, Y_ref, S, dtype, max(abs(alpha), 1.0), np.abs(beta * y0f.astype(np.float64)).reshape(A.m, k), what="fuzz spmm case %d k=%d" % (case, k))
    b200sp.b200sp_check()
