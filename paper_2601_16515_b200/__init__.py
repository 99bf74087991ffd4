"""B200-native SALAD sparse-linear attention forward (sm_100a CUDA kernels behind a C ABI).

``paper_2601_16515_b200.salad``      ctypes binding of ``libsalad.so`` (same names as the C entry points)
``paper_2601_16515_b200.workloads``  seeded synthetic input generators (no method arithmetic)
``paper_2601_16515_b200.build``      nvcc build of the library for sm_100a

Nothing is imported eagerly: importing the package never loads the CUDA library.
"""
__all__ = ["salad", "workloads", "build"]
