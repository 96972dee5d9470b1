"""B200-native Hybrid Sparse Attention (HSA) forward path.

`paper_2609_34606_b200.hsa` is the thin Python binding over the C-ABI library
(libhsa.so, built from csrc/); `paper_2609_34606_b200.workloads` holds the
seeded synthetic input generators.  Importing the package itself loads nothing
native; importing `.hsa` fails loudly if the library has not been built.
"""
__all__ = ["workloads"]
