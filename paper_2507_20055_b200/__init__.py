"""B200-native DeepPoly back-substitution (C-ABI CUDA library + ctypes binding).

`workloads` (seeded inputs) imports without the CUDA library; `binding`
requires the built library and raises if it is missing.
"""
