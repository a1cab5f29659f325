"""From a routed batch to the per-GPU shards the attention kernels take (host only, no arithmetic of the method).

After the all-to-all of a degree-d node every GPU of the node holds the node's samples at full length with 1/d of
the query heads (paper Sec. 2.1); a GPU's shard is the packed list of the samples of all nodes on its leaf-to-root
chain (paper Sec. 4.1.1). Segments are ordered root first, inside a node by nonincreasing length.
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


def load_cost_coefficients(path=None):
    """The measured compute coefficients shipped with the package (written by ``measure_cost_table`` on a B200 for a
    32q/4kv model with head_dim 128, four levels); returns (tcomp_ns [levels, buckets], the file's metadata)."""
    import json
    from pathlib import Path

    path = Path(path) if path else Path(__file__).resolve().parent / "cost_table_b200.json"
    doc = json.loads(path.read_text())
    return np.asarray(doc["tcomp_ns"], dtype=np.float64), doc


def route_batch(lengths, n_levels, b_tok, prefix_k=8, beam_w=4, monotone=True, hq=32, hkv=4, head_dim=128,
                link_gbs=None, other_ns_per_token=400.0, tcomp_ns=None, seed=0):
    """Cost table -> Algorithm 1 -> per-GPU shards, through the library's host functions.

    link_gbs: bandwidth per level (default: 770 GB/s, the measured NVLink 5 peer copy, at every level above 0);
    other_ns_per_token: non-attention time of one layer per resident token. Returns a dict with the routing
    (level, index, load, tok, feasible), the cost table and the shards."""
    from . import binding as B

    if tcomp_ns is None:
        tcomp_ns, _ = load_cost_coefficients()
        if tcomp_ns.shape[0] < n_levels:
            raise ValueError("the shipped coefficients cover fewer levels than requested")
        tcomp_ns = tcomp_ns[:n_levels]
    if link_gbs is None:
        link_gbs = [0.0] + [770.0] * (n_levels - 1)
    cost = B.nsp_cost_table(lengths, n_levels, hq, hkv, head_dim, tcomp_ns, link_gbs, other_ns_per_token)
    level, index, load, tok, feasible = B.nsp_route_sp_tree(lengths, cost, n_levels, prefix_k, beam_w, b_tok, monotone)
    shards, ids = shards_from_routing(lengths, level, index, n_levels, hq, hkv, seed=seed)
    return {"level": level, "index": index, "load_ns": load, "tok": tok, "feasible": feasible, "cost": cost,
            "shards": shards, "sample_ids": ids}
