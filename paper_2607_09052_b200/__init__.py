"""B200-native COBS decode path: CUDA kernels behind a C-ABI library, a thin
ctypes binding with the same names, and the seeded workload generators.

Importing the package loads nothing native; the first call into
``paper_2607_09052_b200.binding`` loads the shared library and fails loudly if
it has not been built.
"""
