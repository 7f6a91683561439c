"""B200-native CKKS RNS primitive layer (CUDA library + thin Python binding).

The compute lives in ``libckks_b200.so`` (hand-written sm_100a kernels behind
a C ABI, see ``include/ckks_b200.h``).  ``binding`` marshals torch tensors into
that ABI; ``inputs`` holds the seeded synthetic input generators.  Importing
the package does not load the library; the first use of ``binding`` does, and
fails loudly if the library has not been built.
"""
__all__ = ["binding", "inputs", "build"]
