"""B200-native implementation of DART's duplication-aware vision-token reduction step.

The compute path is a C-ABI CUDA library (``csrc/``, declared in ``include/dart.h``); ``dart``
is its thin Python binding and ``workloads`` the seeded synthetic input generators.  Importing
the package loads nothing; the binding loads the library on first use and raises if it is absent.
"""
__all__ = ["dart", "workloads"]
