"""Seeded synthetic workloads for the MiLoRA adapter path.

This package only draws random inputs (tensors and batch structure).  It holds none
of the method's arithmetic, so that both the CPU oracle's callers and the CUDA
library's callers can take their inputs from it without sharing any computation.
"""
from .workloads import (  # noqa: F401
    CONFIGS,
    MODULES,
    Workload,
    get_workload,
    module_dims,
    tensor_seed,
)
