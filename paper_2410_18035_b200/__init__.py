"""MiLoRA adapter-apply hot path for NVIDIA B200 (sm_100a): CUDA library + thin ctypes binding.

The kernels live in csrc/ and are built into libmilora.so by `python -m paper_2410_18035_b200.build`;
`binding.Milora` exposes the C ABI declared in include/milora.h.  There is no CPU implementation.
"""
from .binding import (  # noqa: F401
    ACT_GELU, ACT_IDENTITY, ACT_RATIONAL, ACT_RELU, ACT_TANH,
    MODULES, N_MOD,
    POOL_LAST, POOL_MAX, POOL_MEAN, POOL_SELFATTN,
    Milora, MiloraError, load_library,
)
