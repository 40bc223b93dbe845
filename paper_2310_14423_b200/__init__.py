"""B200-native hot path of the Quadratic Synchronization Rule (local steps, replica averaging, round lengths).

`workloads` describes the synthetic runs; `binding` is the thin ctypes layer over the C-ABI library
(`libqsr.so`, built from `csrc/` by `build.py`).  Nothing here falls back to the CPU: importing
`binding` raises if the CUDA library has not been built.
"""
from . import workloads  # noqa: F401

__all__ = ["workloads"]
