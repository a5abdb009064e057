"""Batched worst-case response-time analysis of GPU-using real-time tasksets on NVIDIA B200.

``taskgen``  seeded synthetic tasksets (inputs only; shared with the CPU oracle's tests)
``binding``  thin ctypes binding of the C-ABI library ``libgcaps_rta.so`` (CUDA, sm_100a)
``build``    compiles the native sources in-tree
"""
__all__ = ["taskgen", "binding", "build"]
