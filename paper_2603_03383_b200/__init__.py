"""B200-native static-tree verification for Medusa-style speculative decoding.

The product is the C-ABI library built from ``csrc/`` (see ``include/mtv.h``);
``binding`` is a thin ctypes layer over it and ``synth`` holds the seeded
synthetic workloads.  Nothing here falls back to a CPU implementation: using
``binding`` without the built CUDA library raises.
"""
__all__ = ["binding", "synth", "build"]
