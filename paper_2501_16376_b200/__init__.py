"""B200-native SwiftPrune pruning pass: a C-ABI CUDA library plus a thin binding.

``paper_2501_16376_b200.binding`` loads the compiled library (and raises if it
is missing: there is no CPU fallback); ``paper_2501_16376_b200.synth`` makes
the seeded synthetic workloads.  Nothing is imported eagerly here.
"""
__all__ = ["binding", "synth", "build"]
