"""B200-native policy-gated block-sparse joint attention (the hot path of RAPID^3's
Sparse-Attention policy): a C-ABI CUDA library for sm_100a plus a thin ctypes binding.

``binding.Context`` exposes the library calls; ``inputs`` holds the seeded synthetic workloads.
The CUDA library is loaded on first use and its absence is an error: there is no CPU path.
"""
from . import inputs  # noqa: F401

__all__ = ["inputs", "binding", "build"]
