"""Natural-compression hot path for NVIDIA B200 (sm_100a): a C-ABI CUDA library
(libnatcomp.so, declared in include/natcomp.h) and this thin binding.

Importing the package loads the built library and fails if it is missing; there is
no CPU fallback.  `workloads` holds the seeded synthetic-input generators.
"""
from . import workloads  # noqa: F401
from .binding import *  # noqa: F401,F403
from .binding import EXPORTS, LIB_PATH, NatcompError, P_INF, lib, status_string  # noqa: F401
