"""B200-native decode hot path of delta-prefetched sparse MLP inference.

``binding`` wraps the C-ABI library (``libnp.so``); ``synth`` holds the seeded
workload generators.  Nothing is imported eagerly so that the generators can be
used on machines without the compiled library.
"""
__all__ = ["binding", "synth", "build"]
