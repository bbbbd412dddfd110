"""B200-native majority-vote sparse DSGD step (arXiv 2011.06495, Algorithm 1).

`binding` is the thin ctypes layer over the C-ABI library (include/mv_sparse.h);
`workloads` holds the seeded synthetic input generators; `build` compiles the library.
"""
__all__ = ["binding", "workloads", "build"]
