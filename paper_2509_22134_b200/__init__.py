"""B200-native draft-tree pass of Group Tree Optimization (hand-written CUDA, C ABI).

Importing the package loads nothing native; `paper_2509_22134_b200.binding` loads the
CUDA library and fails loudly if it has not been built.
"""
