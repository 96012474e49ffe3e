"""CPU oracle for the Group Tree Optimization draft-tree pass.

TEST INFRASTRUCTURE ONLY.  This package is the slow, plain fp64 statement of what
the CUDA library computes.  Only the tests, the smoke check and the benchmark's
CPU-baseline leg may import it; the product path never does, and nothing in here
imports the product package.
"""
