"""B200-native MXFP8 conversion and block-scaled GEMM (arXiv 2506.08027), C-ABI + thin binding.

``from paper_2506_08027_b200 import binding`` loads ``libmxfp8.so`` (built in-tree by
``paper_2506_08027_b200.build``); importing the package alone loads nothing, so the input
generators in ``synth`` stay usable without the CUDA library.
"""
__all__ = ["binding", "build", "synth"]
