"""B200-native Winograd convolution with a pre-inference planner.

``workloads`` holds the seeded synthetic layers; ``binding`` is the thin ctypes
face of the C-ABI library (loaded on first use, never at import).
"""
__all__ = ["workloads", "binding"]
