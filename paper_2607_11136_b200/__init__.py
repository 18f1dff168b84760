"""B200-native (sm_100a) library for memory-budgeted DiT blocks: a lifetime trace, a static
arena layout (Algorithm 1), the smallest sequence-chunk count that fits a byte budget, and
the chunked block / denoising step itself as hand-written CUDA kernels behind a C ABI.

`binding` mirrors the C ABI one to one; `session` holds the device buffers (through torch)
that a forward call needs.  Nothing in this package computes on the CPU.
"""
from . import binding  # noqa: F401

__all__ = ["binding"]
