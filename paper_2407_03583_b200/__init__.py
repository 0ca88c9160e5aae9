"""B200-native allocation search of Loki's Resource Manager (HPDC '24).

``workloads`` holds the seeded input generators; ``binding`` is the thin
Python front end of the C-ABI CUDA library ``libloki_alloc.so``.
"""
from . import workloads  # noqa: F401
