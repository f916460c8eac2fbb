"""B200-native decode hot path of KNN-SSD self-speculative decoding.

``binding`` wraps the C-ABI CUDA library (libknnssd.so, built by ``build``); ``metrics`` holds the
host-side reporting formulas.  Importing ``binding`` fails if the library has not been built: there is
no CPU fallback.
"""
__all__ = ["binding", "build", "metrics"]
