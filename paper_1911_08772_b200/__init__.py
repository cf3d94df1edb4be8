"""Error-compensated Gaussian_k gradient sparsifier and exact Top_k for B200.

The compute lives in the CUDA library (csrc/, C ABI declared in include/gk.h);
`binding` marshals arguments to it.  `workloads` holds seeded input generators.
Nothing is loaded at import time; the first call into `binding` loads the
library and raises if it is missing.
"""
__all__ = ["binding", "workloads"]
