"""B200-native LSAM worker step (arXiv 2509.03110): Python binding of the C-ABI CUDA library.

Importing the package is cheap and needs no GPU; the shared library is loaded on first use
and every entry point fails loudly when it is missing (there is no CPU fallback).
"""
from . import synth  # noqa: F401

__all__ = ["synth"]
