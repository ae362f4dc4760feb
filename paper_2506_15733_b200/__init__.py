"""B200-native scoring of drafted candidate blocks for SPECS (arxiv 2506.15733).

``inputs`` draws the seeded synthetic tensors; ``binding`` is the thin ctypes
layer over the C-ABI library built from ``csrc/``.  Importing this package does
not load the shared library; the first call into ``binding`` does, and raises if
the library has not been built.
"""
__all__ = ["inputs", "binding"]
