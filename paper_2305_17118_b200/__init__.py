"""B200-native budgeted KV-cache decode attention (Scissorhands, arXiv 2305.17118).

The product is ``lib/libscissorhands.so`` (hand-written sm_100a kernels behind
the C ABI declared in ``include/scissorhands.h``).  ``binding`` is a thin
ctypes layer over it with the same call names; ``workloads`` draws the seeded
synthetic input streams.  Nothing here falls back to a CPU path: importing
``binding`` without the built library (and without nvcc to build it) raises.
"""
__all__ = ["binding", "workloads", "build"]
