"""B200-native implementation of the DynaMo quantized-MoE inference hot path.

The product is the C-ABI library ``libdynamo.so`` (hand-written sm_100a CUDA kernels,
declared in ``include/dynamo.h``); ``binding`` is the thin ctypes layer with the same
names.  Importing this package loads nothing: the library is opened on first use and
a missing library is an error (there is no CPU fallback).
"""

__all__ = ["binding", "workloads"]
