"""BRACE ring aggregation for NVIDIA B200 (sm_100a): CUDA library + thin binding.

``brace``      ctypes binding of the C-ABI library (include/brace.h); loaded lazily,
               raises if the compiled library is missing -- there is no CPU fallback.
``workloads``  seeded synthetic inputs (no aggregation arithmetic).
"""
