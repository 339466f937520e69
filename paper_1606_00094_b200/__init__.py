"""Convolution-layer forward pass for NVIDIA B200 (sm_100a): C-ABI CUDA library + thin binding.

Importing the package does not load the CUDA library; ``paper_1606_00094_b200.binding`` does, and
fails loudly when the library has not been built.
"""
__all__ = ["workloads", "binding", "build"]
