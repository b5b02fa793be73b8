"""B200-native NVFP4 W4A4 linear layer (activation quantize + block-scaled FP4
GEMM with a per-segment global-scale epilogue).

The compute lives in a C-ABI CUDA library (``include/nvfp4.h``); ``binding``
marshals torch tensors into it.  Importing this package does not load the
library; the first call does, and fails loudly if it has not been built.
``synth`` is the seeded input generator (numpy only).
"""

__all__ = ["binding", "synth", "build"]
