"""B200-native cached partial prefill for VLA-Cache (arxiv 2502.02175).

The package holds three things:

* ``synth``   -- seeded synthetic inputs (frames, features, weights). No arithmetic
                 of the method lives there; both the CUDA path and the CPU checker
                 are fed from it.
* ``csrc/``   -- the CUDA kernels and the C-ABI library (``libvlac.so``).
* ``binding`` -- a thin ctypes layer with the same names as the C entry points.

Importing the package does not load the shared library; ``binding`` does, and it
raises if the library is missing (there is no CPU fallback).
"""

__all__ = ["synth", "binding"]
