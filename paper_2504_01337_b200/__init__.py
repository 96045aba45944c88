"""B200-native hot path of collaboration-constrained routing (C2R) for MoE layers.

`inputs`  : seeded synthetic workloads (no method arithmetic).
`binding` : ctypes binding over the C-ABI library `libc2r.so` (imports fail loudly if the
            library has not been built; there is no CPU fallback).
"""
from . import inputs  # noqa: F401

__all__ = ["inputs"]
