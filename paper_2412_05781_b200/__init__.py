"""sdwino on B200: 3x3 stride-1 pad-1 convolution by the Winograd algorithm (sm_100a).

`binding` wraps the C ABI declared in include/sdwino.h; `workloads` holds the seeded synthetic
layer shapes.  Importing `binding` requires the compiled libsdwino.so (see `build`).
"""
from . import workloads  # noqa: F401
from .build import build_library, LIB_PATH  # noqa: F401

__all__ = ["workloads", "build_library", "LIB_PATH"]
