"""B200-native Adam-mini optimizer step (arxiv 2406.16793, Algorithm 1).

binding    ctypes front end of the CUDA library (libadammini.so, C ABI in include/adammini.h)
workloads  model-shaped tensor lists and seeded synthetic inputs
build      in-tree nvcc build of the library for sm_100a
partition  (name, shape) pairs -> tensor descriptors by Algorithm 2 / Algorithm 3
sharding   whole-block sharding of a step over data-parallel ranks (host logic)
"""
from . import binding, partition, sharding, workloads  # noqa: F401
from .binding import AdamMini, AdamMiniError, Partition  # noqa: F401
