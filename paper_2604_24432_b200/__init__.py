"""B200-native forward pass of Kwai Summary Attention (KSA).

The product is the C-ABI shared library built from ``csrc/`` (declared in
``include/ksa.h``); ``binding`` is a thin ctypes layer with the same entry points.
"""
__all__ = ["binding", "synth"]
