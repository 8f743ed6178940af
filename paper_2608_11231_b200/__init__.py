"""B200-native recurrent-layer hot path of hybrid position-independent caching.

The work is done by a C-ABI CUDA library (``csrc/``, built in-tree as
``liblkv.so``); ``binding`` is the thin ctypes layer over it and ``workloads``
holds the seeded synthetic input generators.  Importing the package does not
load the library; the first call does, and raises if it is missing.
"""
__all__ = ["binding", "workloads"]
