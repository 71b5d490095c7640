"""Isomorphic neighbourhood collectives (all-to-all, allgather, irregular all-to-all)
for P virtual processes on a d-dimensional torus, all resident in one GPU's memory.

The work is done by a C-ABI CUDA library (``csrc/``, declared in ``include/iso.h``);
``binding`` marshals arguments into it and ``workloads`` generates seeded inputs.
Nothing is imported eagerly so that the input generators stay usable on a machine
without the compiled library; every call into the collectives fails loudly when the
library is missing.
"""

__all__ = ["binding", "workloads"]
