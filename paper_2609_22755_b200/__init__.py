"""B200-native local attention compute of nested sequence parallelism: packed variable-length causal GQA attention
(forward, backward, backward with tree-level recomputation) for one GPU's share of an SP-tree plan, plus the steps
either side of it.

Modules: :mod:`binding` (ctypes front-end of the C-ABI CUDA library, loaded lazily; no CPU fallback), :mod:`api`
(one object per packed batch), :mod:`workloads` (seeded synthetic inputs, no CUDA dependency), :mod:`planner`
(cost table -> SP-tree routing -> per-GPU shards, through the library's host functions), :mod:`ulysses` (prologue /
epilogue exchange schedule around the attention call), :mod:`measure_cost_table` (profiles the compute
coefficients of the cost model on the GPU at hand), :mod:`build` (nvcc build of the library)."""

__all__ = ["api", "binding", "build", "planner", "ulysses", "workloads"]
