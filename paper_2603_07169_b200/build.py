"""Builds libb200sp.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import glob
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libb200sp.so")
LIB_CHECKED = os.path.join(HERE, "libb200sp_check.so")     # the same sources with -DB200SP_BOUNDS_CHECK
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-shared"]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = glob.glob(os.path.join(CSRC, "*")) + glob.glob(os.path.join(os.path.dirname(HERE), "include", "*.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    """Compile every .cu under csrc/ into libb200sp.so (checked = True: libb200sp_check.so, the build that validates the
    matrix on the device before every compute call) if it is missing or older than its sources."""
    lib = LIB_CHECKED if checked else LIB
    if force or stale(lib):
        nvcc = os.environ.get("NVCC", "nvcc")
        tmp = lib + ".tmp.%d" % os.getpid()
        cmd = [nvcc] + NVCC_FLAGS + (["-DB200SP_BOUNDS_CHECK"] if checked else []) + (["-Xptxas", "-v"] if verbose else []) + ["-o", tmp] + sources()
        subprocess.check_call(cmd)
        os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    import sys
    print(build(force=True, verbose=True, checked="--bounds-check" in sys.argv))
