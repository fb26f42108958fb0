"""B200-native local sparse SYRK: C_L = tril(A * A^T) on CSR input.

The package holds the CUDA kernels behind a C ABI (``csrc/``, ``libspsyrk.so``), a thin
ctypes binding (``binding``) and the seeded synthetic workload generators (``workloads``).

Importing the package loads nothing native.  ``paper_2608_09713_b200.binding`` loads the
CUDA library and raises if it has not been built; there is no CPU fallback.
"""

__all__ = ["binding", "workloads", "build"]
