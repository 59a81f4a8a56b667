"""B200-native two-sided adaptive rounding (GPTQ-2D).

``workloads`` builds seeded synthetic inputs; ``gptq2d`` is the thin ctypes
binding over the C-ABI CUDA library (it raises if the library is not built --
there is no CPU fallback).
"""
__all__ = ["workloads", "gptq2d"]
