"""B200-native gate step of Entropy Adaptive Decoding: Python binding of the C-ABI library.

The CUDA library (``libead_b200.so``, built by ``paper_2502_06833_b200.build``)
does all the work; this package only marshals arguments.  There is no CPU or
PyTorch fallback: importing ``binding`` without the built library raises.
"""
__all__ = ["binding", "build", "vocab_parallel"]
