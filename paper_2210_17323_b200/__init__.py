"""B200-native GPTQ layer solver: thin Python binding over the C-ABI CUDA library.

Importing the package does not load the CUDA library; `paper_2210_17323_b200.binding`
does, and raises if it is missing (there is no CPU fallback).
"""
__version__ = "0.1.0"
