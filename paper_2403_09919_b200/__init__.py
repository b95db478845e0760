"""B200-native ReDrafter speculative decode step (arXiv 2403.09919).

`paper_2403_09919_b200.binding` is the thin ctypes layer over the C-ABI library
(include/redrafter.h); `paper_2403_09919_b200.synth` draws the synthetic inputs.
Importing the package does not load the CUDA library; the binding does, and it
fails loudly when the library has not been built.
"""
__all__ = ["binding", "synth", "build"]
