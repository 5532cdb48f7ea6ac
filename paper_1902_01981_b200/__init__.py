"""B200-native coded tree aggregation (CodedReduce): C-ABI CUDA library plus a thin ctypes binding.

`binding` mirrors include/codedreduce.h; `inputs` holds the seeded synthetic-input generators;
`build` compiles the library in-tree with nvcc for sm_100a.
"""
from . import binding, inputs  # noqa: F401

__all__ = ["binding", "inputs"]
