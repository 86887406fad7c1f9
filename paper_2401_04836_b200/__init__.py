"""const_b200: fused sparse tensor-network contraction trees (CoNST schedules) on one B200.

The package is a thin ctypes binding over `libconst_b200.so` (C ABI in include/const_b200.h).
Every step of the computation runs in the CUDA library; Python only marshals arguments.
"""
from .binding import (  # noqa: F401
    ConstError,
    CsfHandle,
    PlanHandle,
    F32,
    F64,
    STATUS_NAMES,
    const_csf_build,
    const_csf_build_noalloc,
    const_csf_level,
    const_csf_values,
    const_csf_set_bins,
    const_csf_bin_counts,
    const_csf_work_lists,
    const_debug_set,
    const_plan_create,
    const_schedule_check,
    const_schedule_cin,
    const_plan_reduced_order,
    const_plan_family,
    const_plan_set_tensor_stage,
    const_execute,
    const_last_device_status,
    const_destroy,
    const_status_string,
    const_profile_enable,
    const_profile_read,
    library_path,
    load_library,
)
