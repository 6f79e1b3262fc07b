"""SCOPE sparse video attention for B200 (sm_100a).

The package holds the CUDA kernels (``csrc/``), their C-ABI shared library and a
thin ctypes binding (``binding``), plus the seeded synthetic-input generator
(``inputs``).  Importing the package loads nothing native; the library is opened
on the first call into ``binding`` and a missing library is a hard error.
"""

__all__ = ["binding", "inputs", "build"]
