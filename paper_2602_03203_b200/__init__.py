"""B200-native budgeted KV-cache eviction and decode attention (ForesightKV hot path).

``workloads`` holds the seeded synthetic input generators; ``binding`` is the
thin ctypes layer over the C-ABI library built from ``csrc/``.  Importing the
package loads nothing native; ``binding.lib()`` does, and raises if the CUDA
library has not been built.
"""
__all__ = ["workloads", "binding"]
