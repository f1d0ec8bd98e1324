"""B200-native W8A8 transformer-layer forward of ZeroQuant-HERO behind a C ABI (libhero.so).

`hero` is the thin ctypes binding (argument marshalling only); `workloads` draws the seeded
synthetic inputs; `prep` is the offline, host-side weight preparation.  The CUDA library is
loaded on first use and its absence is an error, never a fallback.
"""
from . import workloads  # noqa: F401

__all__ = ["workloads", "hero", "prep", "build"]
