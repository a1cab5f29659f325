"""From a routed batch to the per-GPU shards the attention kernels take (host only, no arithmetic of the method).

After the all-to-all of a degree-d node every GPU of the node holds the node's samples at full length with 1/d of
the query heads (paper Sec. 2.2); a GPU's shard is the packed list of the samples of all nodes on its leaf-to-root
chain (paper Sec. 4.1). Segments are ordered root first, inside a node by nonincreasing length.
"""
from __future__ import annotations

import numpy as np

from . import workloads as W


def shards_from_routing(lengths, level, index, n_levels, hq, hkv, seed: int = 0):
    """One Workload per GPU. hq / hkv: heads of the whole model; a level-l sample appears with hq / 2^l query heads
    and max(1, hkv / 2^l) KV heads (a KV head shared by several GPUs is replicated). Returns (workloads, sample ids
    per GPU in segment order)."""
    lengths = np.asarray(lengths, dtype=np.int64)
    level = np.asarray(level, dtype=np.int64)
    index = np.asarray(index, dtype=np.int64)
    P = 1 << (n_levels - 1)
    shards, ids = [], []
    for p in range(P):
        mine = [j for j in range(len(lengths)) if (p >> level[j]) == index[j] and lengths[j] > 0]
        mine.sort(key=lambda j: (-level[j], -lengths[j], j))
        d = [1 << int(level[j]) for j in mine]
        if any(hq % x for x in d):
            raise ValueError("the SP degree must divide the number of query heads")
        shards.append(W.custom([int(lengths[j]) for j in mine], [hq // x for x in d], [max(1, hkv // x) for x in d],
                               seed=seed + p, name=f"routed_shard_gpu{p}"))
        ids.append(mine)
    return shards, ids
