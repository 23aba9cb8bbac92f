"""B200 (sm_100a) compressed-sensing attention (CSAT) forward: a C-ABI CUDA library and its binding.

`workloads` (seeded synthetic inputs) imports nothing heavy; `binding` loads libcsat.so and
needs torch + a CUDA device for anything beyond loading.
"""
__all__ = ["workloads", "binding", "build", "autograd"]
