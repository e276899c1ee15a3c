"""B200-native tree-verification step of ConFu-style speculative decoding.

`binding` holds the thin ctypes layer over the C-ABI library (libconfu.so, built
from csrc/ for sm_100a); `inputs` the seeded synthetic workloads.  Nothing here
computes on the CPU: every call fails loudly if the CUDA library is missing.
"""
__all__ = ["binding", "inputs", "build"]
