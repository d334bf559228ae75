"""B200-native DD-EF-SGD / DeCo-SGD hot path: error-feedback Top-k compression, stale
aggregation and apply, as CUDA kernels (sm_100a) behind the C-ABI library ``libdeco``.

``binding`` holds the ctypes wrappers of the C entry points (same names); ``workloads`` the
seeded synthetic inputs.  Nothing is loaded at import time.
"""
