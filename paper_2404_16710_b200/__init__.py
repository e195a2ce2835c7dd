"""B200-native batch-1 self-speculative greedy decoding (LayerSkip, arXiv 2404.16710, Sec. 4.3).

``paper_2404_16710_b200.binding`` is the thin ctypes layer over the C-ABI CUDA
library (``libls_b200.so``, built in-tree from ``csrc/``); ``synth`` draws the seeded
synthetic inputs.  Importing the package loads nothing; the first use of the
binding loads the library and fails loudly if it is missing.
"""
__all__ = ["binding", "synth"]
