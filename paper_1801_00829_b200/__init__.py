"""Fused-operator execution (Cell, MAgg, Row, Outer templates) on one B200 GPU.

The work happens in ``libfusedops.so`` (CUDA, sm_100a; C ABI in
``include/fusedops.h``; test and measurement hooks in ``include/fusedops_tools.h``); this package is the thin ctypes binding around it.
"""
from .binding import (  # noqa: F401
    CSR, FusedOpsError, cell_stamps, chain_describe, device_status, force_interpreter, fused_cell, fused_cell_static, fused_magg, fused_outer, fused_row, fused_row_b1,
    jit_compile_check, jit_compile_check_outer, jit_compile_check_row, jit_prepare, jit_prepare_call, jit_stats, load_library, make_chain, probe_bulk_flag_index, probe_bulk_gather, probe_fp64_fma, probe_l2_gather, probe_out_len, set_jit, tune,
    workspace,
)
from .roofline import (  # noqa: F401
    algorithmic_bytes, ideal_seconds, operator_cost, operator_sizes, plan_cost, unfused_plan_sizes,
)

__all__ = [
    "CSR", "FusedOpsError", "cell_stamps", "chain_describe", "device_status", "force_interpreter", "fused_cell", "fused_cell_static", "fused_magg", "fused_outer",
    "fused_row", "fused_row_b1", "jit_compile_check", "jit_compile_check_outer", "jit_compile_check_row", "jit_prepare", "jit_prepare_call", "jit_stats", "set_jit", "load_library", "make_chain", "workspace", "algorithmic_bytes", "ideal_seconds", "operator_cost", "operator_sizes", "plan_cost", "unfused_plan_sizes",
    "probe_bulk_flag_index", "probe_bulk_gather", "probe_fp64_fma", "probe_l2_gather", "probe_out_len", "tune",
]
