"""B200 (sm_100a) library for the target-side verify step of Mirror Speculative Decoding.

`binding` wraps the C-ABI CUDA library (include/mirror.h); `inputs` draws the seeded synthetic
workloads.  Importing this package loads nothing; the library is loaded on first use and there is
no fallback if it is missing.
"""
__all__ = ["binding", "inputs"]
