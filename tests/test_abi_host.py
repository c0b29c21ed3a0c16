"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the header
declares, and rejects bad arguments before touching the device."""
import ctypes
import os
import re

import numpy as np
import pytest

import paper_2603_07169_b200 as b200sp
from paper_2603_07169_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = "".join(open(os.path.join(ROOT, "include", f)).read() for f in sorted(os.listdir(os.path.join(ROOT, "include"))) if f.endswith(".h"))
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"\b([a-z_0-9]+)\s*\(", text)
    return sorted({n for n in names if n.startswith(("spmv_", "spmm_", "b200sp_"))})


def test_library_exports_every_declared_symbol():
    L = b200sp.lib()
    names = declared_functions()
    assert len(names) >= 16
    for n in names:
        assert hasattr(L, n), "libb200sp.so does not export %s" % n
    assert set(names) == set(binding.EXPORTS)      # the binding wraps exactly the declared entry points


def test_version_and_strings():
    assert b200sp.b200sp_version() >= 100
    L = b200sp.lib()
    for s in range(0, 8):
        assert L.b200sp_status_string(s) not in (None, b"")


BAD = 1  # B200SP_ERR_INVALID_ARG


def test_invalid_arguments_are_rejected_on_the_host():
    L = b200sp.lib()
    buf = np.zeros(64, np.int32)
    p = buf.ctypes.data           # numpy data is 16-byte aligned or better here
    assert p % 16 == 0
    # negative sizes
    assert L.spmv_csr(-1, 4, 0, p, p, p, p, p, 1.0, 0.0, 0, None) == BAD
    assert L.spmv_csr(4, -1, 0, p, p, p, p, p, 1.0, 0.0, 0, None) == BAD
    assert L.spmv_csr(4, 4, -1, p, p, p, p, p, 1.0, 0.0, 0, None) == BAD
    # sizes past int32
    assert L.spmv_csr(4, 4, 1 << 31, p, p, p, p, p, 1.0, 0.0, 0, None) == BAD
    # unknown dtype
    assert L.spmv_csr(4, 4, 4, p, p, p, p, p, 1.0, 0.0, 7, None) == BAD
    # NULL pointers with non-zero sizes
    assert L.spmv_csr(4, 4, 4, None, p, p, p, p, 1.0, 0.0, 0, None) == BAD
    assert L.spmv_csr(4, 4, 4, p, None, p, p, p, 1.0, 0.0, 0, None) == BAD
    assert L.spmv_csr(4, 4, 4, p, p, p, p, None, 1.0, 0.0, 0, None) == BAD
    # misaligned operand
    assert L.spmv_csr(4, 4, 4, p, p + 4, p, p, p, 1.0, 0.0, 0, None) == BAD
    assert L.spmv_csr(4, 4, 4, p, p, p, p + 2, p, 1.0, 0.0, 1, None) == BAD
    # SpMM: k <= 0
    assert L.spmm_csr(4, 4, 4, 0, p, p, p, p, p, 1.0, 0.0, 0, None) == BAD
    assert L.spmm_csr(4, 4, 4, -3, p, p, p, p, p, 1.0, 0.0, 0, None) == BAD
    # nnz > 0 in a matrix without rows or columns
    assert L.spmv_csr(0, 4, 4, p, p, p, p, p, 1.0, 0.0, 0, None) == BAD
    # host variants validate the same way
    assert L.spmv_csr_host(4, 4, 4, p, p, p, p, p, 1.0, 0.0, 9, None) == BAD
    assert L.spmm_csr_host(4, 4, 4, 0, p, p, p, p, p, 1.0, 0.0, 0, None) == BAD
    # plan API
    out = ctypes.c_void_p()
    assert L.b200sp_plan_create(None, 4, 4, 4, p, None) == BAD
    assert L.b200sp_plan_create(ctypes.byref(out), 4, 4, 4, None, None) == BAD
    assert L.b200sp_spmv(None, p, p, p, p, 1.0, 0.0, 0, None) == BAD
    assert L.b200sp_plan_info(None, None) == BAD
    assert L.b200sp_set_option(b"no_such_option", 1) == BAD
    assert L.b200sp_set_option(b"spmv_kernel", 5) == BAD
    assert L.b200sp_set_option(b"row_unroll", 3) == BAD


def test_switches_read_back_and_environment_at_load():
    """b200sp_get_option returns what b200sp_set_option stored; B200SP_OPTIONS / B200SP_LOG in the environment set switches when
    the library is loaded (checked in a process of its own), and an entry that is not accepted is reported and skipped."""
    import subprocess
    import sys
    assert b200sp.b200sp_get_option("merge_items") == 2048
    b200sp.b200sp_set_option("merge_items", 4096)
    try:
        assert b200sp.b200sp_get_option("merge_items") == 4096
    finally:
        b200sp.b200sp_set_option("merge_items", 2048)
    with pytest.raises(b200sp.B200spError):
        b200sp.b200sp_get_option("no_such_option")
    code = ("import sys; sys.path.insert(0, %r); import paper_2603_07169_b200 as b; "
            "print(b.b200sp_get_option('spmv_kernel'), b.b200sp_get_option('merge_short'), b.b200sp_get_option('log'), b.b200sp_get_option('row_unroll'))" % ROOT)
    env = dict(os.environ, B200SP_OPTIONS="spmv_kernel=0,merge_short=16,row_unroll=5,nonsense", B200SP_LOG="1")
    out = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True, env=env, timeout=120)
    assert out.returncode == 0, out.stderr
    assert out.stdout.split() == ["0", "16", "1", "8"]
    assert "row_unroll=5" in out.stderr and "nonsense" in out.stderr


def test_empty_problem_is_a_no_op_without_a_device():
    L = b200sp.lib()
    assert L.spmv_csr(0, 0, 0, None, None, None, None, None, 1.0, 0.0, 0, None) == 0
    assert L.spmm_csr(0, 5, 0, 3, None, None, None, None, None, 1.0, 0.0, 1, None) == 0


def test_binding_raises_with_status():
    with pytest.raises(b200sp.B200spError) as e:
        b200sp.spmv_csr(-1, 0, 0, None, None, None, None, None, 1.0, 0.0, "f32", stream=0)
    assert e.value.status == BAD


def test_device_entry_points_refuse_host_arrays_before_anything_is_launched():
    """A numpy array (or a CPU tensor) handed to a device entry point would make a kernel dereference a host address; the
    binding refuses it with INVALID_ARG and the library is never entered."""
    import torch
    n0 = b200sp.b200sp_launch_count()
    a = np.zeros(64, np.int32)
    f = np.zeros(64, np.float32)
    for bad in (a, torch.zeros(64, dtype=torch.int32)):
        with pytest.raises(b200sp.B200spError) as e:
            b200sp.spmv_csr(4, 4, 4, bad, a, f, f, f, 1.0, 0.0, "f32", stream=0)
        assert e.value.status == BAD
    with pytest.raises(b200sp.B200spError) as e:
        b200sp.spmm_csr(4, 4, 4, 8, a, a, f, f, f, 1.0, 0.0, "f32", stream=0)
    assert e.value.status == BAD
    with pytest.raises(b200sp.B200spError) as e:       # host entry point: too short an array is refused as well
        b200sp.spmv_csr_host(100, 100, 400, a, a, f, f, f, 1.0, 0.0, "f32", stream=0)
    assert e.value.status == BAD
    assert b200sp.b200sp_launch_count() == n0


def test_product_path_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2603_07169_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower(), "%s mentions the oracle" % f
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".c")):
            text = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2603_07169_b200" not in text and "libb200sp" not in text
