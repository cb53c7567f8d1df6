"""HilbertA sparse attention forward for B200 (sm_100a).

The compute lives in the C-ABI shared library built from csrc/ (see
include/hilberta.h); `binding` is the thin ctypes layer over it, and `inputs`
holds the seeded synthetic workloads.  Nothing here computes on the CPU.
"""
__version__ = "0.1.0"
