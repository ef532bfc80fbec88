"""B200-native fused dequantize-plus-matvec over Leech-lattice (Lambda24(12)) quantised weights.

`binding` mirrors the C ABI of include/llvq.h; `datagen` draws the seeded synthetic inputs; `build`
compiles the CUDA library in-tree.  Importing the package loads nothing: the shared library is
loaded by the first binding call, which raises if it has not been built.
"""
from . import binding, datagen  # noqa: F401

__all__ = ["binding", "datagen"]
