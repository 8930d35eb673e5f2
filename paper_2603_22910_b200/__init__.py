"""B200-native EchoKV decode attention: CUDA kernels behind a C-ABI, with a thin ctypes binding.

Importing the package loads nothing native; `paper_2603_22910_b200.binding` loads the
shared library and fails loudly if it has not been built.
"""
