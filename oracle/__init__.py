"""CPU oracle for the SmoothQuant W8A8 hot path (test infrastructure only).

Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this package; the CUDA library and its binding never do.
"""
from .sq_oracle import *  # noqa: F401,F403
from . import sq_oracle as _m

__all__ = [n for n in dir(_m) if not n.startswith("_")]
