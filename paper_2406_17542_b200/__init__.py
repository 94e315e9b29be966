"""B200-native CDQuant hot path: greedy coordinate-descent weight quantization.

The compute lives in a C-ABI CUDA library (``include/cdq.h``); ``binding``
marshals torch tensors into it and ``inputs`` draws the synthetic layers.
Importing this package loads nothing; the library is loaded on first call.
"""
__all__ = ["binding", "inputs"]
