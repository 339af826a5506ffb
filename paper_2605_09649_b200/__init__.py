"""B200-native decode hot path of global retention-based KV eviction.

`binding` wraps the C-ABI library (CUDA kernels, sm_100a); `workloads` draws seeded
synthetic inputs.  There is no CPU fallback: using `binding` without the built shared
library raises.
"""
__all__ = ["binding", "workloads"]
