"""B200-native melded FP8-LoRA linear layer (forward, backward, row-wise proxy update).

The compute lives in hand-written CUDA kernels for sm_100a behind a C-ABI
shared library (``libfalqon.so``, declared in ``include/falqon.h``);
``paper_2510_24061_b200.binding`` marshals arguments to it and nothing else.
"""
