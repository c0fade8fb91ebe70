"""VMoBA block-sparse attention hot path for NVIDIA B200 (sm_100a).

The product is the C-ABI library ``libvmoba.so`` built from ``csrc/``; ``binding``
is a thin ctypes layer over it (argument marshalling only) and ``inputs`` holds the
seeded synthetic-input generators.  Importing this package does not load the library;
``binding.lib()`` does, and raises if the library has not been built.
"""
__all__ = ["inputs", "binding", "build"]
