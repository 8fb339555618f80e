"""Seeded synthetic inputs (operand matrices and fault-site tables).

This package only draws numbers and lays them out in storage format. It holds
none of the GEMM, injection or detection arithmetic, so both the CPU oracle's
tests and the CUDA path's tests can use it without sharing method code.
"""
from .generators import (config_seed,   # noqa: F401
    DTYPE_FP16, DTYPE_BF16, DTYPE_TF32,
    KIND_A, KIND_B, KIND_ACC, KIND_OUT, KIND_TERM,
    SITE_DTYPE, CONFIGS, Workload,
    kstep, storage_dtype, round_to_storage, make_operands, make_sites,
    make_workload, adjacent_mask,
)
