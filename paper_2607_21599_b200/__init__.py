"""B200-native (sm_100a) implementation of the DAF prefill-attention path.

`paper_2607_21599_b200.api` is the Python binding of the C-ABI library declared
in include/daf.h; `paper_2607_21599_b200.workloads` holds the seeded synthetic
inputs.  Importing the package does not load the CUDA library; the first call
into `api` does, and raises if the library is missing.
"""
__all__ = ["api", "workloads"]
