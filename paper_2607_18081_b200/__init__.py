"""SelectInfer selective-FFN hot path for B200 (sm_100a).

``paper_2607_18081_b200.api`` is the thin binding over the C-ABI CUDA library
(``libselectinfer.so``); ``paper_2607_18081_b200.workloads`` makes the seeded synthetic
inputs.  Importing the package loads neither torch nor the CUDA library.
"""
__all__ = ["api", "workloads"]
