"""B200-native local-layer training step of adaptive local learning (NeuroFlux, arXiv 2402.14139).

``nf`` is the thin binding over the C-ABI library ``libnf.so``; ``synth`` holds the seeded input
generators.  Importing ``nf`` fails loudly when the CUDA library has not been built.
"""
