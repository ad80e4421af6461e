"""B200-native (sm_100a) KVCache retrieval hot path: page scoring, per-head top-k, cluster
resolution with queue balancing, gather and split-K sparse attention, behind a C-ABI library.

``binding`` holds the ctypes binding (same names as the C entry points); ``workloads`` holds
the seeded synthetic input generators.  Nothing here falls back to a CPU implementation:
calling an op without the compiled CUDA library raises.
"""
__all__ = ["binding", "workloads", "build"]
