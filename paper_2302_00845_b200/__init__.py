"""B200-native PairBalance ordering library for CD-GraB (arXiv 2302.00845).

The product is the C-ABI shared library built from ``csrc/`` (declared in
``include/cdgrab.h``); ``binding`` is a ctypes layer with the same names.
"""
__all__ = ["binding", "synth", "build"]
