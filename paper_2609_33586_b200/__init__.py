"""Rowmax-H15 / Rowmax-PoT / exact fused attention forward for B200 (sm_100a).

``inputs`` holds the seeded synthetic workloads; ``binding`` is the thin ctypes layer over the
C-ABI library (``include/attn.h``) that runs every step of the path in CUDA kernels.
"""
__all__ = ["inputs", "binding"]
