"""MGRIT solve of the GRU recurrence on one B200: Python binding of the C-ABI library.

Importing the package does not load the CUDA library; `paper_2203_04738_b200.binding`
does, and fails loudly if it has not been built.
"""
