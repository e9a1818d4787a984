"""B200-native hot path of DSpark's serving step: the confidence-scheduled
verification-length scheduler and the fused ragged-batch speculative verifier.

``paper_2607_05147_b200.binding`` is the thin ctypes layer over the C-ABI
library built from ``csrc/``; ``workloads`` holds the seeded synthetic inputs.
"""
__all__ = ["binding", "workloads", "build"]
