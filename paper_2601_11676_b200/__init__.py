"""B200-native group-sparse FFN hot path of HALO (arXiv 2601.11676).

``binding`` is the thin ctypes layer over the C-ABI library ``libhalo.so``;
``synth`` holds the seeded synthetic workloads.  Importing the package loads
no native code; ``binding.lib()`` does, and fails loudly if the library has
not been built.
"""
__all__ = ["binding", "synth", "build"]
