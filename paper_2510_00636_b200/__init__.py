"""Expected Attention KV-cache scoring and pruning for NVIDIA B200 (sm_100a).

The product is a C-ABI shared library of hand-written CUDA kernels
(``include/ea.h``); :mod:`paper_2510_00636_b200.binding` marshals torch tensors
into it.  Importing this package does not load the library; the first call
does, and fails loudly when the library has not been built.
"""
__all__ = ["binding", "inputs", "build"]
