"""Ternary Weight Networks hot path for NVIDIA B200 (sm_100a).

`paper_1605_04711_b200.twn` binds the C-ABI CUDA library; `datagen` draws the
seeded synthetic tensors used by tests and benchmarks.  Importing the package
loads nothing; the CUDA library is opened on first use and its absence is an
error, never a fallback.
"""
