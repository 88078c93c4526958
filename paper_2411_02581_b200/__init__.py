"""TuNA (tunable-radix non-uniform all-to-all) hot path for NVIDIA B200.

``workloads`` holds the seeded input generators; ``binding`` is the thin
ctypes layer over the C-ABI library built from ``csrc/`` (it raises if the
library is missing: there is no CPU fallback).
"""
__all__ = ["workloads", "binding", "build"]
