"""B200-native row-typed associative-algebra projection (Y = X *_q W) and FFN.

The compute lives in the CUDA library ``libalgproj.so`` (C ABI, see ``include/algproj.h``);
``binding`` is the thin ctypes layer above it and ``synth`` the seeded input generators.
Nothing is loaded at import time; ``binding.lib()`` raises if the library has not been built.
"""
__all__ = ["binding", "synth"]
