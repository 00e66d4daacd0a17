"""B200-native sufficient-factor hot path (factor computation, SF buffer, rank-K apply).

`binding` mirrors the C ABI of include/sfb.h; `workload` puts a synthetic workload on the device.
The CUDA library must be built (`build.build_library()`); nothing here computes on the CPU.
"""
from . import binding
from .build import build_library, LIB_PATH

__all__ = ["binding", "build_library", "LIB_PATH"]
