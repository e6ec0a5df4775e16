"""B200-native sparse denoising step of a world-action model's joint attention (Sparse-WAM).

`workloads` holds shapes and the seeded synthetic generator; `swam` is the
binding of the CUDA library (libswam.so), loaded on first use.
"""
from . import workloads  # noqa: F401

__all__ = ["workloads"]
