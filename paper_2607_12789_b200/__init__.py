"""B200-native AVQ-attention forward (adaptive vector-quantized attention).

The compute lives in a C-ABI CUDA library (``include/avq_attn.h``); ``binding``
marshals torch tensors into it.  Importing the package does not load the
library; the first call that needs it does, and fails loudly if it is missing.
"""
__all__ = ["synth", "binding", "build"]
