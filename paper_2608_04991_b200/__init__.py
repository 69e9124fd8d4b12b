"""B200-native hot path of the RAC reference-aware activation codec.

``synth`` draws the seeded workloads; ``binding`` is the thin ctypes layer over
the C-ABI library ``librac.so`` (CUDA kernels for sm_100a).  Nothing here falls
back to a CPU implementation: the binding raises when the library is missing.
"""
__version__ = "0.1.0"
