"""B200-native clustered-head attention (CHAI, arXiv 2403.08058): C-ABI CUDA library + thin binding.

Importing the package does not load the CUDA library; the first call through
``paper_2403_08058_b200.chai`` does, and raises if it has not been built.
"""
__all__ = ["chai", "synth"]
