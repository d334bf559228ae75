"""CPU oracle for the DD-EF-SGD / DeCo-SGD hot path — TEST INFRASTRUCTURE ONLY.

Plain, slow, obviously-correct restatement of what the paper's Algorithm 1 (DD-EF-SGD),
Algorithm 3 (DeCo) and Theorem 3 (iteration-time model) compute.  It shares no code with the
CUDA library and must never be imported by the product package: only ``tests/``, the smoke
check and the benchmark's CPU-baseline / reference legs use it.
"""
