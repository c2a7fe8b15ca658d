"""B200-native chunked instruction-aware state eviction (CItruS hot path).

`workloads` draws synthetic inputs; `binding` is the thin ctypes layer over the
C-ABI library built from `csrc/`.  Nothing here computes on the CPU.
"""
from . import workloads  # noqa: F401

__all__ = ["workloads", "binding"]
