"""B200-native decode step of a GTM-constrained SID generator (GRACE).

Thin ctypes binding over libgrace_b200.so: argument marshalling only.  Every
step of the path runs in the library's CUDA kernels; there is no CPU or
framework fallback, and importing `paper_2608_00938_b200.api` raises if the
library has not been built.
"""
from .build import build  # noqa: F401

__all__ = ["build", "api"]
