"""B200-native DQ-SGD gradient quantizer hot path (arXiv 2107.14575).

``paper_2107_14575_b200.dq``        thin ctypes binding of the C-ABI CUDA library
``paper_2107_14575_b200.workloads`` seeded synthetic gradient generators

Importing the package loads nothing; the binding loads ``libdq.so`` on first
use and raises if it has not been built.
"""
__all__ = ["dq", "workloads"]
