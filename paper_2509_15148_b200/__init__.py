"""B200-native ATTS verification hot path: fused LM-head scoring + conformal rejection.

The CUDA library is loaded on first use of :mod:`paper_2509_15148_b200.binding`;
importing the package (or its input generators) needs no GPU.
"""
__all__ = ["inputs"]
