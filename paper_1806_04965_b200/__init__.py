"""Streaming-rollout frame update on B200: Python binding of the C-ABI CUDA library.

The package holds the CUDA sources (csrc/), their build step (build.py) and a thin
ctypes binding (binding.py) with the same names as the C entry points.  Every step
of the frame update runs in the library's kernels; Python only marshals arguments.
"""
from .binding import Graph, SrError, load_library, STATUS  # noqa: F401
