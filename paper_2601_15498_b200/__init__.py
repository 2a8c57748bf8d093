"""B200-native margin-aware speculative verification (MARS).

``mars``  -- ctypes binding of the C-ABI CUDA library (argument marshalling only).
``synth`` -- seeded synthetic workloads (input construction only).
``build`` -- nvcc build of the library for sm_100a.

Importing the package loads nothing; the shared library is opened on the first call
into ``mars`` and a missing library is an error, never a fallback.
"""
__all__ = ["mars", "synth", "build"]
