"""EOQ full 8-bit integer training layer (arXiv 2105.13890) on sm_100a.

``eoq`` is the thin binding over the C-ABI library (``include/eoq.h``); ``synth``
holds the seeded synthetic input generators and ``workloads`` the layer-shape
lists of the benchmark networks.  The CUDA library is loaded on first use and
there is no CPU fallback: a missing library raises.
"""
__all__ = ["eoq", "synth", "workloads"]
