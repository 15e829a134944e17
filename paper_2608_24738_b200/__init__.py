"""B200-native exact Euclidean distance transform (``tm_edt``).

``binding`` is the thin ctypes layer over the C-ABI CUDA library; ``workloads`` holds the seeded
synthetic inputs.  Importing the package loads nothing native: the CUDA library is opened on first use
and its absence is an error, never a fallback.
"""
__all__ = ["binding", "workloads", "buildlib"]
