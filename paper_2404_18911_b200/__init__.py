"""B200-native (sm_100a) implementation of the Kangaroo batch-1 self-speculative decode step.

`binding` is a thin ctypes layer over the C ABI in include/kangaroo.h (libkangaroo.so, built
in-tree by `build.build()`); every step of the method runs in the CUDA kernels.
"""
from .build import build as build_library, lib_path  # noqa: F401
