"""Paged attention over a dynamically FP8-quantised KV cache with grouped-query sharing,
as hand-written sm_100a CUDA kernels behind a C-ABI library (``libcoopt.so``).

``workloads`` draws seeded synthetic inputs; ``binding`` marshals torch tensors into
the C calls.  Nothing here computes on the CPU: if the shared library is missing the
binding raises instead of falling back.
"""
__all__ = ["workloads", "binding", "build"]
