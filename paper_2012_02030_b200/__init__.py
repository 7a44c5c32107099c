"""Attention Pruning's compute path for NVIDIA B200: a C-ABI CUDA library
(csrc/, declared in include/ap.h) plus a thin ctypes binding (binding.py).

`inputs` (seeded synthetic workloads) and `metrics` (host-side counters) import
without the CUDA library; `binding` needs libap_b200.so and fails without it.
"""
