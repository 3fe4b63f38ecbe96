"""B200-native W4A16 (group-wise INT4 weight-only) linear layer: AWQ's inference hot path.

The compute lives in the C-ABI CUDA library built from ``csrc/``; ``binding`` marshals
torch tensors into its calls.  Importing the package does not load the library; the
first call does, and fails loudly if it has not been built.
"""
__all__ = ["binding", "synth", "build"]
