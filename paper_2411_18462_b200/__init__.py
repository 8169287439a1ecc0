"""SVIP speculative-decoding epilogues for NVIDIA B200 (sm_100a).

The work is done by hand-written CUDA kernels behind the C ABI declared in
``include/svip.h``; this package only loads that library and marshals
arguments (``binding``), builds it (``build``) and generates the seeded
synthetic workloads (``workloads``).  There is no CPU fallback: without the
compiled library every call raises.
"""
from .binding import (  # noqa: F401
    SVIP_BF16, SVIP_F32, SVIP_Q_PACKED, Context, Graph, SvipError, library, library_path, verify_noalloc,
)

__all__ = ["SVIP_BF16", "SVIP_F32", "SVIP_Q_PACKED", "Context", "Graph", "SvipError", "library",
           "library_path", "verify_noalloc"]
