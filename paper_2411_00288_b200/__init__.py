"""2:4 semi-structured sparse convolution for B200 (sm_100a).

The hot path is a C-ABI CUDA library (see include/ssconv.h); `api` is its thin ctypes
binding and `synth` draws the seeded synthetic workloads.  Importing the package does
not load the library; the first call through `api` does, and fails loudly if it has
not been built.
"""
__all__ = ["api", "synth", "build"]
