"""Paged decode attention for B200 (sm_100a): RoPE + KV append, split-KV attention, LSE merge.

The CUDA kernels live behind the C ABI declared in ``include/ac.h``; ``binding`` is the thin ctypes
layer with the same names.  Importing the package does not load the shared library; the first call
through ``binding`` does, and raises if it has not been built.
"""
__all__ = ["binding", "workloads", "build"]
