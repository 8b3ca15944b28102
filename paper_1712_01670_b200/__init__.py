"""DeepCache hot path on B200: block matcher, region propagation, partial convolution.

The CUDA library is loaded on first use (``paper_1712_01670_b200.binding``);
importing the package, or its ``synth`` input generators, does not need a GPU.
"""
__all__ = ["binding", "synth"]
