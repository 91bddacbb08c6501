"""B200-native block-sparse decode attention of Elastic Threshold Attention.

The product is the C-ABI library built from `csrc/` (see `include/eta.h`);
`binding` is its thin ctypes front end, `workloads` the seeded input
generators used by tests and benchmarks.
"""
