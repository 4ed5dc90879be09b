"""CoreInfer core-sparse FFN path for NVIDIA B200 (sm_100a).

`binding` is the ctypes front of the C-ABI library (include/coreinfer.h); `workloads`
holds the seeded synthetic input generators; `_build` compiles the CUDA sources in-tree.
"""
from . import _build, binding, pipeline, workloads  # noqa: F401
from .binding import *  # noqa: F401,F403
