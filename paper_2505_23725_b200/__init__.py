"""B200-native MuLoCo optimizer step: a CUDA library (libmuloco.so, built from
csrc/) behind a C ABI (include/muloco.h) and a thin ctypes binding.

Importing the package does not load the library; `binding.load_library()` (or
constructing `binding.MuLoCo`) does, and raises if it has not been built.
"""
from . import configs, synth  # noqa: F401

__all__ = ["configs", "synth", "binding", "build"]
