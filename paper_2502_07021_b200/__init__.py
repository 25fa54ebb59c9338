"""B200-native Sinkhorn hot path (row / column kernel-operator passes, log-domain passes,
shared-K batched passes) behind the C-ABI library ``libfs_b200.so``.

``workloads`` holds the seeded input generators; ``binding`` the ctypes layer over the C ABI.
Importing the package does not load the CUDA library; ``binding.lib()`` does, and raises if
it has not been built.
"""
from . import workloads  # noqa: F401

__all__ = ["workloads"]
