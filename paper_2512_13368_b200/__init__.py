"""B200-native BlossomRec block-sparse attention (long-term selected blocks +
short-term causal window + learnable gate), forward and backward.

The arithmetic lives in the CUDA library behind a C ABI (``include/blossom.h``);
this package is the thin ctypes binding plus seeded synthetic workloads.
"""
from . import workloads  # noqa: F401  (numpy only; no CUDA needed)

__all__ = ["workloads"]
