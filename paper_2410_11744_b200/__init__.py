"""B200-native tree-verify attention (DySpec, Sec. 2 "Tree Attention"): C-ABI CUDA library + thin binding.

Importing the package does not load the CUDA library; `paper_2410_11744_b200.binding` does, and fails
loudly if it has not been built.
"""
__all__ = ["workloads"]
