"""B200-native spectral-split NVFP4 linear layer (Metis): thin Python binding over the C-ABI library.

Importing the package does not load the CUDA library; `paper_2509_00404_b200.binding` does, and
raises if the library has not been built.  There is no CPU fallback.
"""
__all__ = ["synth"]
