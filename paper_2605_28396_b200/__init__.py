"""B200-native windowed on-policy-distillation divergence path (ADWIN hot path).

The compute lives in the CUDA shared library built from ``csrc/``; ``api`` is the thin ctypes
binding with the same entry-point names, ``synth`` the seeded input generators.  Importing the
package does not load the library; the first call through ``api`` does and fails loudly when the
library is missing.
"""
__all__ = ["api", "synth", "build"]
