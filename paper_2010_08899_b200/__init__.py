"""B200-native (sm_100a) kernels for the Dynamic Communication Thresholding compression path.

The product is the C-ABI library declared in ``include/dct.h``; :mod:`.binding`
marshals torch tensors into it.  The shared library is loaded on first use and
its absence is an error: there is no CPU or PyTorch fallback.
"""
__all__ = ["binding", "inputs", "build"]
