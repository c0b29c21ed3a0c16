"""b200sp: CSR SpMV / SpMM for NVIDIA B200 behind a C ABI (libb200sp.so).

The Python layer only marshals arguments (see ``binding``); the product is the CUDA library built
from ``csrc/`` and declared in ``include/b200sp.h`` (tuning switches and probes: ``include/b200sp_tuning.h``).
"""
from .binding import (BF16, F32, B200spError, b200sp_cache_clear, b200sp_cache_drop, b200sp_check, b200sp_launch_count, b200sp_plan_create,  # noqa: F401
                      b200sp_plan_destroy, b200sp_plan_info, b200sp_set_option, b200sp_get_option, b200sp_spmm, b200sp_spmv,
                      b200sp_validate_csr, b200sp_version, b200sp_checked_build, lib, spmm_csr, spmm_csr_host, spmv_csr, spmv_csr_host,
                      spmv_csr_noalloc, b200sp_noalloc_max_items, b200sp_probe_gather, b200sp_probe_gather_ex, b200sp_probe_stream, b200sp_probe_lines, b200sp_probe_spmv_gather, b200sp_spmv_naive, b200sp_spmm_naive, spmv_coo, spmm_coo, spmv_ell, spmm_ell, spmv_csc, spmm_csc, spmv_csr_vec_host)
