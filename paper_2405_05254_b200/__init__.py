"""B200-native cross-decoder attention over the shared K/V cache (YOCO, Section 2.2).

The product is the C-ABI library built from ``csrc/`` (declared in ``include/yoco_xattn.h``);
``binding`` is a thin ctypes layer with the same entry-point names.  Importing this package does
not load the CUDA library; ``binding`` loads it on first use and fails loudly when it is missing.
"""
__all__ = ["binding", "build"]
