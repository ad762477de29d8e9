"""B200-native block-quantised prefill GEMM (dense and mixture-of-experts).

The compute path is a C-ABI CUDA library for sm_100a (see include/qgemm.h); `binding` is its thin
ctypes wrapper and is loaded lazily, so importing the package (or `synth`, the seeded input
generators) needs neither a GPU nor the built library.
"""
__all__ = ["synth", "binding"]
