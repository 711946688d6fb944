"""B200-native multi-tenant MoE layer (FaaSMoE hot path) behind a C-ABI CUDA library.

``workloads`` holds the seeded input generators; ``binding`` the ctypes
front-end of ``libfaasmoe.so`` (loaded on first use, never a CPU fallback).
"""
__all__ = ["workloads", "binding", "build"]
