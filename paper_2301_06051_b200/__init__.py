"""DSVT dynamic sparse window attention for NVIDIA B200: hand-written CUDA behind a C ABI.

`api` is the ctypes binding (same names as include/dsvt.h); `build` compiles the library in-tree.
Importing this package loads nothing; `api.load()` / `api.Context` load the shared library and
raise if it has not been built.
"""
from . import api  # noqa: F401
