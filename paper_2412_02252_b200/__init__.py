"""PoD decode attention over a compressed KV cache, hand-written CUDA for sm_100a.

The product is the C-ABI library declared in ``include/pod.h``; ``binding`` wraps it with
the same names.  ``synth`` is the seeded input generator shared by tests and bench.
"""
