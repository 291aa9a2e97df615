"""B200-native FastSGD gradient compression / decompression (arxiv 2112.04291).

The hot path lives in hand-written CUDA kernels behind a C-ABI shared library
(``libfastsgd_b200.so``, declared in ``include/fastsgd.h``); ``binding`` is the thin
ctypes layer with the same names.  Importing this package does not load the library;
``binding`` does, and raises if it is missing: there is no CPU fallback.
"""
__all__ = ["binding", "workloads", "build"]
