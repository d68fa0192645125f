"""B200-native hot path of Neural Garbage Collection (score, sample, log-prob,
compact, ragged decode attention) behind a C-ABI CUDA library.

``paper_2604_18002_b200.binding`` holds the thin Python binding (argument
marshalling only); ``paper_2604_18002_b200.synth`` the seeded input generators.
Nothing here falls back to the CPU: importing ``binding`` without the built
CUDA library raises.
"""
__all__ = ["binding", "synth"]
