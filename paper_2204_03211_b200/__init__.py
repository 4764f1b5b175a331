"""Packed model aggregation for Parameter Service on one B200.

The product is the C-ABI library declared in include/ps_b200.h (CUDA kernels
for sm_100a under csrc/); `binding` is its ctypes face.  There is no CPU or
library fallback: without the built .so every call raises.
"""
from . import binding  # noqa: F401
from .binding import Service, Planner, PsError  # noqa: F401
