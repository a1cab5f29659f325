"""B200-native packed variable-length causal GQA attention (forward + backward) for one GPU's share of a
nested sequence-parallel plan. The CUDA library is loaded lazily by :mod:`paper_2609_22755_b200.binding`;
:mod:`paper_2609_22755_b200.workloads` (seeded synthetic inputs) has no CUDA dependency."""

__all__ = ["binding", "workloads", "build"]
