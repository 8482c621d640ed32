"""B200-native SLoPe 2:4-sparse linear layer (hand-written sm_100a kernels behind a C ABI).

``inputs`` (seeded synthetic tensors) imports without the CUDA library;
``binding`` loads ``libslope.so`` and fails loudly when it is missing.
"""
__all__ = ["inputs", "binding", "build"]
