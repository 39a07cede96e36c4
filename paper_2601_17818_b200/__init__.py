"""B200-native visual-token pruning operator chain of ViTCoP (arXiv 2601.17818).

The product is the C-ABI library built from ``csrc/`` (declared in ``include/vitcop.h``);
``binding`` is a thin ctypes layer with the same entry-point names, and ``workloads``
holds the seeded synthetic input generators.
"""
__version__ = "0.1.0"
