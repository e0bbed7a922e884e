"""B200-native hot path of a predictive multi-tier KV-cache manager.

The CUDA library (libkvtier.so, built from csrc/) is loaded on first use by
`paper_2604_26968_b200.binding`; `workloads` only draws synthetic inputs.
"""
__all__ = ["binding", "workloads"]
