"""PRAC per-linear-layer activation compression for B200 (sm_100a).

The computation lives in libprac.so (hand-written CUDA, C ABI declared in include/prac.h);
this package is a thin ctypes binding with the same names plus the seeded synthetic input
generators.  There is no CPU or PyTorch fallback: importing `api` without the built
library raises.
"""
from . import inputs  # noqa: F401

__all__ = ["inputs", "api", "build"]
