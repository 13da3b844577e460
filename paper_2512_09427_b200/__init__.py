"""B200-native slab-KV decode attention for ODMA (on-demand contiguous KV allocation).

The package holds the CUDA/C++ sources of the C-ABI library (`csrc/`), its thin
ctypes binding (`odma`) and the seeded synthetic inputs (`workloads`).  Importing
the package loads nothing; `paper_2512_09427_b200.odma` loads the shared library
and raises if it has not been built.
"""
__all__ = ["odma", "workloads", "build"]
