"""B200-native batched evaluation of rematerialization sequences (Moccasin, arXiv 2304.14463).

``paper_2304_14463_b200.binding`` is the thin ctypes layer over the C-ABI CUDA library;
``paper_2304_14463_b200.workloads`` generates seeded synthetic inputs.  Nothing is imported
eagerly, so the input generators can be used without the CUDA library.
"""
__all__ = ["binding", "workloads"]
