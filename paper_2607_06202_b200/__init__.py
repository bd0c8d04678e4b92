"""B200-native MoE token dispatch / combine with virtual expert-parallel ranks.

``binding`` is the thin ctypes layer over the C-ABI CUDA library (same names as the C
entry points); ``workload`` holds the seeded input generators.  Importing the package
loads nothing native; the first call into ``binding`` loads the library and fails
loudly if it has not been built.
"""
__all__ = ["binding", "workload"]
