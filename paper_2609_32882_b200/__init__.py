"""B200-native VSA2 routed block-sparse attention (forward and backward).

The compute lives in the CUDA library built from ``csrc/``; ``binding`` marshals
arguments into its C ABI.  Importing the package does not load the library, so the
input generators stay usable on a machine without a GPU; every operator call fails
loudly if the library is missing.
"""
