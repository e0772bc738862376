"""Shift-accumulate decode attention for B200 (sm_100a): Python binding of the C-ABI library.

The package holds the CUDA sources (``csrc/``), their build step (``build.py``), the thin
ctypes binding (``binding.py``) and the seeded input generators (``synth.py``).  Importing
the package does not load the CUDA library; ``binding.lib()`` does, and raises if it is missing.
"""
__all__ = ["synth", "binding", "build"]
