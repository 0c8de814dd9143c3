"""DyBit quantize/pack and coded-operand GEMM/conv for NVIDIA B200 (sm_100a).

The product is the C-ABI library ``libdybit.so`` (see ``include/dybit.h``);
this package is its ctypes binding plus synthetic workload generators.
"""
from .binding import *  # noqa: F401,F403
from .binding import __all__ as _binding_all
from . import workloads  # noqa: F401

__all__ = list(_binding_all) + ["workloads"]
