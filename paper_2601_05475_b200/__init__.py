"""Shared-prefix (cascade) grouped-query decode attention over a paged KV cache for B200 (sm_100a).

`workload` draws the seeded synthetic inputs; `binding` is the thin ctypes layer over the C-ABI
library built from `csrc/` (every step of the path runs in that library's CUDA kernels).
"""
