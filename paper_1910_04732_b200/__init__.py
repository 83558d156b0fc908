"""B200-native hot path of FLOP (factorized low-rank pruning): the gated
factorized linear layer W = P diag(z) Q with hard-concrete L0 gates.

`inputs` holds the seeded synthetic workloads; `binding` is the thin ctypes
layer over the C-ABI CUDA library (it raises if the library is missing: there
is no CPU fallback).
"""
__all__ = ["inputs", "binding"]
