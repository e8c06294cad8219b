"""Decode attention over a KV cache split between GPU HBM and pinned host
memory, for NVIDIA B200 (sm_100a).

The compute lives in ``libisv.so`` (CUDA, C ABI, declared in ``include/isv.h``);
``binding`` marshals arguments for it and ``workloads`` holds seeded synthetic
inputs.  Importing this package does not load the library; the first call that
needs it does, and fails loudly if it has not been built.
"""
__all__ = ["binding", "workloads"]
