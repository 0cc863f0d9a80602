"""B200-native step attention for KV-cache reuse with contiguous RoPE.

The compute path lives in the C-ABI library ``libevln.so`` (CUDA, sm_100a); ``binding``
is the thin ctypes layer over it and ``workloads`` draws the seeded synthetic inputs.
Nothing here falls back to the CPU: importing ``binding`` fails loudly when the library
has not been built.
"""
__all__ = ["workloads", "binding"]
