"""B200-native ZGR step (zeroth-order optimisation with cloud-guided gradient rectification).

``paper_2601_12917_b200.zgr`` is the thin ctypes binding of the C ABI declared in
``include/zgr.h``; the CUDA kernels live in ``csrc/``.  ``paper_2601_12917_b200.synth`` holds
the seeded synthetic inputs.  Importing the package loads nothing; the shared library is
loaded on first use and its absence is an error (there is no CPU fallback).
"""
__all__ = ["zgr", "synth"]
