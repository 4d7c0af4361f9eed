"""B200-native (sm_100a) hot path of the FEPLB per-micro-batch MoE layer.

``paper_2604_19654_b200.feplb`` is the thin binding over the C-ABI library ``libfeplb.so``
(routing histogram, rebalancing plan, dispatch permutation, grouped SwiGLU expert FFN on
tcgen05/TMEM, gated combine); ``paper_2604_19654_b200.workloads`` draws the seeded synthetic
inputs.  Importing the package loads nothing: the library is opened on first use and its
absence is an error, never a fallback.
"""
__all__ = ["feplb", "workloads"]
