"""B200-native decode attention over a line-structured compressed KV cache (LineAR hot path).

`paper_2512_04857_b200.lar` is the thin ctypes binding of the C-ABI library (CUDA kernels, sm_100a);
`paper_2512_04857_b200.workloads` holds the synthetic workload shapes and the seeded input generator.
Importing the package does not load the CUDA library; `lar.lib()` does, and raises if it is missing.
"""
__all__ = ["workloads", "lar"]
