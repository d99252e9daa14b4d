"""B200-native hot path of a HADFL training round (arXiv 2111.08274).

`binding` wraps the C-ABI library (CUDA kernels for sm_100a); `workloads` holds the seeded
synthetic inputs.  Nothing here falls back to a CPU implementation: using the binding without
the built library raises.
"""
__all__ = ["binding", "workloads", "build"]
