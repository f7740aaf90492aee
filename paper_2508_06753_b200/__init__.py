"""B200-native W2A8 (2-bit weight x int8 activation) GEMV/GEMM hot path.

``synth`` holds the seeded input generators; ``binding`` is the thin ctypes
layer over the C-ABI CUDA library (``libw2a8.so``).  Importing the package
does not load the library; ``binding.lib()`` does, and fails loudly when it
is missing.
"""
__all__ = ["synth", "binding"]
