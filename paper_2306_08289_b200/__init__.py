"""A2CiD2 event-update engine for one B200: CUDA kernels behind a C ABI, plus a thin binding.

Importing the package loads nothing native; `paper_2306_08289_b200.binding` loads the shared
library on first use and raises if it is missing (there is no CPU fallback)."""

__all__ = ["workload", "binding", "build"]
