"""B200-native PEQA quantized-linear hot path (arXiv 2305.14152).

The compute lives in hand-written sm_100a CUDA kernels behind a C-ABI shared
library (see ``include/peqa.h``).  ``binding`` marshals torch tensors into that
ABI; ``synth`` draws the seeded inputs.  Importing the package does not load
the library; the first call through ``binding`` does, and fails loudly if the
library has not been built.
"""
__all__ = ["binding", "synth", "build"]
