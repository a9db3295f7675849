"""B200-native CoCoD-SGD parameter engine (arxiv 1906.12043, Algorithm 1).

``engine``  : thin ctypes binding over the C-ABI library ``libcocod.so`` (CUDA, sm_100a)
``inputs``  : seeded synthetic inputs (no method arithmetic)

Nothing here falls back to the CPU: using the engine without the built CUDA
library raises.
"""
__all__ = ["engine", "inputs"]
