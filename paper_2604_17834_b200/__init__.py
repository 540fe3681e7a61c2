"""B200-native SpMM (BCSR and WCSR) -- hand-written sm_100a CUDA behind a C ABI.

``paper_2604_17834_b200.binding`` is the thin ctypes layer over the shared
library; ``paper_2604_17834_b200.workloads`` draws the seeded synthetic
inputs.  Importing the package does not load the CUDA library; the binding
does, and it fails loudly when the library is missing.
"""
__all__ = ["binding", "workloads", "build"]
