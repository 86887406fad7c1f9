"""Seeded synthetic inputs shared by the tests, the oracle checks and the benchmark.

This package only draws random tensors and writes down schedule descriptors. It
contains none of the contraction or CSF arithmetic: both the CUDA library and the
CPU oracle receive its arrays as plain inputs.
"""
from .generators import (  # noqa: F401
    Workload,
    CONFIG_NAMES,
    make_config,
    ttmc3_workload,
    ttmc4_workload,
    mttkrp_workload,
    network_workload,
    zipf_slice_sizes,
    row_sample,
)
