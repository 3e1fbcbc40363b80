"""Full-memory random cache-line reads on B200 (arXiv 2405.11425), as a C-ABI CUDA library.

`binding` exposes the entry points of include/rr.h one to one; `pipeline` strings them into the
paper's experiments (size sweep, pair probe, clustering, grouped windows).
"""
from .binding import *  # noqa: F401,F403
from .binding import _load as _load_library

__all__ = [n for n in dir() if n.startswith(("rr_", "RR_", "Read"))]
