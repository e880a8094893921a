"""Importance-weighted gradient pruning for data-parallel all-reduce, native to B200.

`paper_1901_01544_b200.binding` is the thin ctypes layer over the C-ABI library
(`include/iwp.h`); `paper_1901_01544_b200.workloads` holds the seeded synthetic
inputs.  Importing the package has no side effects and needs no GPU.
"""
