"""B200-native decode hot path of a three-tier (full / low-bit recoverable / deleted) window KV cache.

The compute lives in hand-written sm_100a CUDA kernels behind a C-ABI shared
library (`libqevict.so`, declared in include/qevict.h); `binding` is the thin
ctypes layer over it and `workloads` draws seeded synthetic inputs.
"""

__all__ = ["binding", "workloads"]
