"""TEST INFRASTRUCTURE — the CPU oracle for the paged FP8 GQA attention path.

Plain, slow, float64 / bit-level definitions written from the paper.  Only ``tests/``,
the smoke check and the benchmark's CPU-baseline leg may import this package.  It shares
no code with the CUDA path and never imports it.
"""
from . import e4m3, kv_cache, attention  # noqa: F401
