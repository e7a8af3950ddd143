"""B200-native batched builder and evaluator of KV-memory-constrained inference schedules.

``workloads`` holds the seeded input generators (no scheduling arithmetic); ``binding`` is the
ctypes front end of the CUDA library declared in ``include/kvs.h``; ``api`` allocates outputs.
The CUDA library is loaded on first use and there is no CPU path.
"""
from . import workloads  # noqa: F401

__all__ = ["workloads", "binding", "api", "build"]
