"""B200-native On-Demand-Attention decode path: thin Python binding over the C-ABI
library (paper_2609_20734_b200.binding) and the seeded input generator (synth)."""
__all__ = ["binding", "synth", "workloads"]
