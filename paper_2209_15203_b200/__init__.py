"""B200-native compression pipeline of bidirectional top_K SGD (arXiv 2209.15203).

``binding`` loads the CUDA library (C ABI in ``include/topk.h``) through ctypes;
``workloads`` holds the seeded synthetic inputs.  Importing the package loads
nothing: the CUDA library is opened on first use and raises if it is missing.
"""
__all__ = ["binding", "workloads"]
