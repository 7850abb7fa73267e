"""B200-native random-walk + SGNS hot path (GraphScale node-embedding training).

`paper_2407_15452_b200.binding` is the thin ctypes layer over the C-ABI library
(`include/gs.h`); `paper_2407_15452_b200.workloads` holds the seeded synthetic
inputs.  Importing the package loads nothing native; the binding loads the
shared library on first use and raises if it has not been built.
"""
__all__ = ["binding", "workloads", "build", "replicas"]
