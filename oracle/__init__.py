"""CPU fp64 oracle for the Hybrid Sparse Attention (HSA) forward path.

TEST INFRASTRUCTURE ONLY.  Nothing in the product package imports this; it is
called from the tests, from the smoke check and from the benchmark's CPU
baseline / reference arm.  It shares no code with the CUDA path.
"""
