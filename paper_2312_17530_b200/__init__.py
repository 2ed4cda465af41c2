"""B200-native RS-DGC gradient compression (arxiv 2312.17530): C-ABI CUDA library + binding.

``paper_2312_17530_b200.binding`` loads the CUDA library and exposes the C entry points;
``paper_2312_17530_b200.synth`` holds the seeded synthetic inputs.  Importing the package
itself loads nothing, so the input generators can be used without a GPU.
"""
__all__ = ["binding", "synth"]
