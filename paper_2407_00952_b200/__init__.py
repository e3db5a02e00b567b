"""B200-native split-LoRA round (arxiv 2407.00952): C-ABI CUDA library + thin binding.

Importing the package loads nothing heavy; `binding` loads the shared library on
first use and raises if it is missing (there is no CPU fallback).
"""
__all__ = ["synth", "binding", "build"]
