"""DEER-GRU hot path for B200 (sm_100a): C-ABI CUDA library + thin binding.

Importing the package does not load the CUDA library; ``binding`` does, and
fails loudly if it is missing.  ``synth`` holds the seeded input generators.
"""
__all__ = ["binding", "synth"]
