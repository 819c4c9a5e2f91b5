"""SkipDecode decode path for B200: CUDA kernels behind a C ABI, plus a thin binding.

Importing the package loads nothing; `paper_2307_02628_b200.binding` opens the
shared library on first use and raises if it has not been built.
"""
__all__ = ["binding", "shapes", "synth", "build"]
