"""B200-native fused AdaGC + AdamW optimizer step (Algorithm 1 of arXiv 2502.11034).

`paper_2502_11034_b200.binding` is the thin ctypes layer over the C ABI declared in
include/adagc.h; every step of the path runs in the CUDA kernels of csrc/ (one translation unit, adagc.cu).
Importing the package loads nothing; the first use of the binding loads libadagc.so and
fails loudly if it has not been built (there is no CPU fallback).
"""
from . import workloads  # noqa: F401

__all__ = ["workloads", "binding", "sharded", "build"]
