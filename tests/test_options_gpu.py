"""Every tuning switch that b200sp_set_option accepts selects shipped CUDA code, so every accepted value of every switch
is run here against the CPU oracle, element by element, on three small matrices (power-law, uniform 16 per row,
27-point stencil) in both dtypes; the switches of the SpMM kernels on SpMM problems with many and with few columns.
The kernel a switch belongs to is forced where the plan would not pick it, so that the switch is really exercised."""
import numpy as np
import pytest

import gen
import paper_2603_07169_b200 as b200sp
from gpu_util import assert_within, run_spmm, run_spmv

pytestmark = pytest.mark.gpu

DEFAULTS = {
    "spmv_kernel": -1, "x_l2_window": 0, "pdl": 1,
    "row_unroll": 8, "row_threads": 256, "row_stages": 2, "row_ctas": 3, "row_smem_kb": 220,
    "uni_unroll": 0, "uni_ctas": 0, "sub_lanes": 0,
    "merge_items": 2048, "merge_threads": 128, "merge_short": 32, "merge_carve": 45, "merge_empty": 0,
    "spmm_bstage": 1, "spmm_sliced": 1, "spmm_ranges": 1, "spmm_stage_a": 2, "spmm_flat": 2, "bstage_threads": 1024, "bstage_nnz": 0, "bstage_stage_a": 1, "bstage_quads": 1,
}

# (switch, accepted values, SpMV kernel to force so that the switch matters; None = leave the choice to the plan)
SPMV_SWITCHES = [
    ("x_l2_window", [0, 1], None),
    ("pdl", [0, 1], None),
    ("spmv_kernel", [-1, 0, 1, 2, 3], None),
    ("row_unroll", [8, 16], 1), ("row_threads", [128, 256], 1), ("row_stages", [2, 3, 4], 1), ("row_ctas", [1, 2, 3, 4], 1),
    ("row_smem_kb", [48, 96, 160, 220, 227], 1),
    ("uni_unroll", [0, 1, 2, 4], 2), ("uni_ctas", [0, 1, 2, 4, 8], 2),
    ("sub_lanes", [0, 1, 2, 4, 8, 16, 32], 3),
    ("merge_items", [1024, 2048, 4096], 0), ("merge_threads", [64, 128, 256], 0), ("merge_short", [8, 16, 32, 64], 0),
    ("merge_carve", [-1, 0, 25, 45, 60, 75, 100], 0), ("merge_empty", [0, 1], 0),
]
SPMM_SWITCHES = [
    ("x_l2_window", [0, 1]), ("pdl", [0, 1]), ("spmm_bstage", [0, 1]), ("spmm_sliced", [0, 1]), ("spmm_ranges", [0, 1, 2, 3, 4, 8]), ("spmm_stage_a", [0, 1, 2]), ("spmm_flat", [0, 1, 2]),
    ("bstage_threads", [256, 512, 1024]), ("bstage_nnz", [0, 16384, 65536, 131072, 524288]), ("bstage_stage_a", [0, 1]), ("bstage_quads", [0, 1]),
]


def spmv_matrices():
    rng = np.random.default_rng(21)
    lens = (rng.pareto(1.2, 6000) * 3).astype(np.int64).clip(0, 3500)
    lens[::7] = 0
    return {
        "power_law": gen.random_csr(6000, 4000, lens, seed=3),
        "uniform16": gen.uniform_rows(6001, 5000, 16, 4),
        "stencil27": gen.stencil27(14, 6),
    }


def reset_all():
    for name, v in DEFAULTS.items():
        b200sp.b200sp_set_option(name, v)


def cases(table):
    out = []
    for entry in table:
        for v in entry[1]:
            out.append((entry[0], v) + tuple(entry[2:]))
    return out


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("switch,value,force", cases(SPMV_SWITCHES), ids=lambda c: str(c))
def test_spmv_switch_value_against_oracle(switch, value, force, dtype):
    rng = np.random.default_rng(5)
    try:
        if force is not None:
            b200sp.b200sp_set_option("spmv_kernel", force)
        b200sp.b200sp_set_option(switch, value)
        for name, A in spmv_matrices().items():
            x = rng.standard_normal(A.n).astype(np.float32)
            y0 = rng.standard_normal(A.m).astype(np.float32)
            y, y_ref, S = run_spmv(A, x, None, 1.0, 0.0, dtype)
            assert_within(y, y_ref, S, dtype, what="%s=%d %s %s" % (switch, value, name, dtype))
            y, y_ref, S = run_spmv(A, x, y0, -0.75, 0.5, dtype, use_plan=True)
            y0f = y0 if dtype == "f32" else gen.bf16_to_f32(gen.to_bf16(y0))
            assert_within(y, y_ref, S, dtype, 1.0, np.abs(0.5 * y0f.astype(np.float64)), what="%s=%d %s %s ab" % (switch, value, name, dtype))
        b200sp.b200sp_check()
    finally:
        reset_all()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("switch,value", cases(SPMM_SWITCHES), ids=lambda c: str(c))
def test_spmm_switch_value_against_oracle(switch, value, dtype):
    rng = np.random.default_rng(6)
    try:
        b200sp.b200sp_set_option(switch, value)
        # few columns (the shape that keeps a slice of B in shared memory) and many columns (the k-sliced kernel), sorted columns
        for m, n, k in ((3000, 2048, 64), (3000, 2048, 40), (4000, 30000, 64), (4000, 30000, 24)):
            lens = rng.integers(0, 40, m)
            lens[3] = min(n, 3000)
            lens[4] = 400
            A = gen.random_csr(m, n, lens, seed=m + k, sort_cols=True)
            B = rng.standard_normal(n * k).astype(np.float32)
            Y0 = rng.standard_normal(m * k).astype(np.float32)
            Y, Y_ref, S = run_spmm(A, B, k, None, 1.0, 0.0, dtype)
            assert_within(Y, Y_ref, S, dtype, what="%s=%d n=%d k=%d" % (switch, value, n, k))
            Y, Y_ref, S = run_spmm(A, B, k, Y0, 1.5, -0.5, dtype)
            y0f = Y0 if dtype == "f32" else gen.bf16_to_f32(gen.to_bf16(Y0))
            assert_within(Y, Y_ref, S, dtype, 1.5, np.abs(0.5 * y0f.astype(np.float64)).reshape(m, k), what="%s=%d n=%d k=%d ab" % (switch, value, n, k))
        b200sp.b200sp_check()
    finally:
        reset_all()


def test_every_switch_of_the_header_is_covered_here():
    """The list of switches in include/b200sp_tuning.h and the tables above must name the same switches (the test switches
    spin_limit / debug_no_copies / fail_alloc_after, pool_keep_mb and log have tests of their own)."""
    import os
    import re
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    text = open(os.path.join(root, "include", "b200sp_tuning.h")).read()
    declared = set(re.findall(r'^ \*\s+"([a-z_0-9]+)"', text, flags=re.M))
    elsewhere = {"spin_limit", "debug_no_copies", "fail_alloc_after", "pool_keep_mb", "log"}
    here = {s[0] for s in SPMV_SWITCHES} | {s[0] for s in SPMM_SWITCHES}
    assert declared == here | elsewhere, (sorted(declared - here - elsewhere), sorted((here | elsewhere) - declared))
    assert set(DEFAULTS) == here
    # a value outside a switch's list is refused
    for name, values in [(s[0], s[1]) for s in SPMV_SWITCHES + SPMM_SWITCHES]:
        bad = max(values) + 1
        if name in ("x_l2_window", "pdl", "spmm_bstage", "spmm_sliced", "bstage_stage_a", "bstage_quads", "merge_empty"):
            continue        # booleans: any non-zero value means 1
        with pytest.raises(b200sp.B200spError):
            b200sp.b200sp_set_option(name, bad)
    reset_all()
