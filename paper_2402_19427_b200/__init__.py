"""RG-LRU temporal core (Conv1D(4) + gates + log-space decay + linear recurrence) for NVIDIA B200.

``inputs`` holds the seeded synthetic workloads (numpy only); ``binding`` is the thin ctypes
layer over the C-ABI CUDA library and is imported lazily so that the input generators can be
used without loading the library.
"""
__all__ = ["inputs", "binding"]
