"""B200 (sm_100a) learner library for GALA-A2C (arXiv 1906.04585).

`binding` exposes the C ABI of include/gala.h one to one; `build` compiles
libgala.so in-tree.  Importing this package loads nothing: the shared library
is opened on first use and its absence is an error, never a fallback.
"""
from . import binding, build  # noqa: F401

__all__ = ["binding", "build"]
