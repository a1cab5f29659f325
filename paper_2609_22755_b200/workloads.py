"""Seeded synthetic workloads: segment lengths, per-segment head counts and bf16 tensors.

This module holds none of the method's arithmetic. It is the one module that both the CUDA tests/bench and
the CPU oracle's tests consume, so that both sides see the same bytes.

A workload is one GPU's share of a nested sequence-parallel plan (paper Sec. 4.1.1, Def. 1 and the per-GPU
leaf-to-root chain): a packed list of segments, each at its own Ulysses degree d, which after the all-to-all
appears on this GPU at full length with H/d query heads (paper Sec. 2.1). The five named configurations and
their scaled-down twins follow the benchmark definition; lengths are long-tailed like the paper's corpora
(Sec. 3.1, Fig. "long-tail": 94.0 % of samples below 8K tokens), drawn from a lognormal.

Recipe for lognormal lengths: x = median * exp(sigma * z), z ~ N(0,1) from numpy PCG64(seed);
L = 16 * max(1, floor(x / 16 + 0.5)); clip to [lo, hi]; L = min(L, remaining budget); stop when the budget is
used up (so the last segment may be shorter than lo).
Tensor values: iid N(0,1) from torch's CPU generator (manual_seed(seed)), rounded to bf16 (RNE),
drawn in the order Q, K, V, dO.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

HEAD_DIM = 128


@dataclass
class Workload:
    name: str
    cu_seqlens: np.ndarray  # int32 [n_seg + 1]
    hq: np.ndarray  # int32 [n_seg]
    hkv: np.ndarray  # int32 [n_seg]
    head_dim: int = HEAD_DIM
    seed: int = 0
    note: str = ""
    extra: dict = field(default_factory=dict)

    @property
    def n_seg(self) -> int:
        return len(self.hq)

    @property
    def lengths(self) -> np.ndarray:
        return np.diff(self.cu_seqlens).astype(np.int64)

    @property
    def softmax_scale(self) -> float:
        return 1.0 / float(np.sqrt(self.head_dim))

    def q_elems(self) -> int:
        return int((self.lengths * self.hq).sum() * self.head_dim)

    def kv_elems(self) -> int:
        return int((self.lengths * self.hkv).sum() * self.head_dim)

    def lse_elems(self) -> int:
        return int((self.lengths * self.hq).sum())

    def q_offsets(self) -> np.ndarray:
        return np.concatenate([[0], np.cumsum(self.lengths * self.hq * self.head_dim)]).astype(np.int64)

    def kv_offsets(self) -> np.ndarray:
        return np.concatenate([[0], np.cumsum(self.lengths * self.hkv * self.head_dim)]).astype(np.int64)

    def lse_offsets(self) -> np.ndarray:
        return np.concatenate([[0], np.cumsum(self.lengths * self.hq)]).astype(np.int64)

    def causal_pairs(self) -> int:
        """sum over segments of Hq * L(L+1)/2 (query/key pairs inside the causal mask)."""
        L = self.lengths
        return int((self.hq.astype(np.int64) * (L * (L + 1) // 2)).sum())

    def flops(self):
        """(forward, backward) FLOPs with exact causal pairs: 4*D and 10*D per (pair, q head)."""
        p = self.causal_pairs()
        return 4 * self.head_dim * p, 10 * self.head_dim * p

    def algorithmic_bytes(self, dkv_bytes: int = 4, dq_bytes: int = 2) -> int:
        """HBM bytes fwd+bwd must move at least once: fwd reads Q,K,V, writes O,LSE; bwd reads
        Q,K,V,O,dO,LSE, writes dQ,dK,dV, plus the delta vector written and read once."""
        qe, kve, le = self.q_elems(), self.kv_elems(), self.lse_elems()
        fwd = 2 * (qe + 2 * kve) + 2 * qe + 4 * le
        bwd = 2 * (3 * qe + 2 * kve) + 4 * le + dq_bytes * qe + 2 * dkv_bytes * kve + 8 * le
        return fwd + bwd


def lognormal_lengths(seed: int, budget: int, median: float, sigma: float, lo: int, hi: int) -> list[int]:
    rng = np.random.Generator(np.random.PCG64(seed))
    out = []
    remaining = budget
    while remaining > 0:
        z = float(rng.standard_normal())
        x = median * np.exp(sigma * z)
        L = 16 * max(1, int(np.floor(x / 16.0 + 0.5)))
        L = min(max(L, lo), hi)
        L = min(L, remaining)
        out.append(L)
        remaining -= L
    return out


def _mk(name, lengths, hq, hkv, seed, note="", head_dim=HEAD_DIM):
    cu = np.concatenate([[0], np.cumsum(np.asarray(lengths, dtype=np.int64))])
    assert cu[-1] < 2**31
    return Workload(name, cu.astype(np.int32), np.asarray(hq, np.int32), np.asarray(hkv, np.int32), head_dim, seed, note)


def config(idx: int, seed: int | None = None, twin: bool = False) -> Workload:
    """The five benchmark configurations (idx 1..5; idx 6 is the mixed-degree shard of `full_tree_shard`) or their scaled-down twins (same head structure,
    lengths divided by 16..32, sized so the fp64 oracle evaluates every element in seconds to a minute)."""
    if seed is None:
        seed = idx - 1
    if idx == 1:
        return _mk("cfg1_tiny", [64, 128, 256, 512], [8] * 4, [2] * 4, seed, "degree 1, GQA 4:1")
    if idx == 2:
        if twin:
            return _mk("cfg2_twin_16x512", [512] * 16, [32] * 16, [4] * 16, seed)
        return _mk("cfg2_static_sp_16x8192", [8192] * 16, [32] * 16, [4] * 16, seed)
    if idx == 3:
        if twin:
            Ls = lognormal_lengths(seed, 4096, 64, 1.3, 16, 2048)
            return _mk("cfg3_twin_longtail_4096", Ls, [32] * len(Ls), [4] * len(Ls), seed)
        Ls = lognormal_lengths(seed, 65536, 1024, 1.3, 16, 32768)
        return _mk("cfg3_longtail_65536", Ls, [32] * len(Ls), [4] * len(Ls), seed)
    if idx == 4:
        if twin:
            short = lognormal_lengths(seed, 1024, 64, 1.2, 16, 512)
            return _mk("cfg4_twin_nested", [12288] + short, [4] + [32] * len(short), [1] + [4] * len(short), seed,
                       "one degree-8 segment + degree-1 tail")
        short = lognormal_lengths(seed, 32768, 2048, 1.2, 64, 16384)
        return _mk("cfg4_nested_shard", [393216] + short, [4] + [32] * len(short), [1] + [4] * len(short), seed,
                   "one 393,216-token segment at degree 8 (4q/1kv) + degree-1 tail (32q/4kv) filling 32,768 tokens")
    if idx == 5:
        if twin:
            short = lognormal_lengths(seed, 4096, 128, 1.0, 16, 2048)
            return _mk("cfg5_twin_largehead", [4096] + short, [16] + [64] * len(short), [1] + [4] * len(short), seed)
        short = lognormal_lengths(seed, 262144 - 131072, 4096, 1.0, 64, 65536)
        return _mk("cfg5_largehead_longtail", [131072] + short, [16] + [64] * len(short), [1] + [4] * len(short), seed,
                   "one 131,072-token segment at degree 4 (16q/1kv) + degree-1 tail (64q/4kv)")
    if idx == 6:
        return full_tree_shard(seed, twin)
    raise ValueError("config index must be 1..6")


def full_tree_shard(seed: int = 5, twin: bool = False) -> Workload:
    """One GPU's chain in a full binary SP tree over eight GPUs (paper Sec. 4.1.1, Def. 1) for a 32q/4kv model: the
    root's segment at degree 8 (4q/1kv), two at degree 4 (8q/1kv), four at degree 2 (16q/2kv) and a long-tailed
    degree-1 leaf batch (32q/4kv). Four runs with four different head counts in one shard. Not one of the five
    benchmark configurations (index 6); the twin divides the lengths by 32."""
    if twin:
        leaf = lognormal_lengths(seed, 1024, 64, 1.2, 16, 512)
        lens = [4096] + [1024, 528] + [256, 304, 128, 200] + leaf
    else:
        leaf = lognormal_lengths(seed, 16384, 1024, 1.2, 64, 8192)
        lens = [131072] + [32768, 16400] + [8192, 9744, 4096, 6160] + leaf
    hq = [4] + [8] * 2 + [16] * 4 + [32] * len(leaf)
    hkv = [1] + [1] * 2 + [2] * 4 + [4] * len(leaf)
    return _mk("full_tree_shard_twin" if twin else "full_tree_shard", lens, hq, hkv, seed,
               "degrees 8 / 4 / 2 / 1 of a 32q/4kv model in one shard")


def profile_case(seed: int = 3) -> Workload:
    """A scaled-down nested shard for profiler captures: one 65,536-token segment at degree 8 (4q/1kv) plus a
    degree-1 tail (32q/4kv) filling 8,192 tokens. About 0.7 GB on the device (more than L2), a few hundred
    milliseconds of kernels even under a multi-pass capture."""
    short = lognormal_lengths(seed, 8192, 2048, 1.2, 64, 16384)
    return _mk("nested_profile_case_64k", [65536] + short, [4] + [32] * len(short), [1] + [4] * len(short), seed,
               "one 65,536-token segment (4q/1kv) + degree-1 tail (32q/4kv) filling 8,192 tokens")


def profile_case_large_head(seed: int = 4) -> Workload:
    """The large-head shard at one eighth of its size, for profiler captures: one 16,384-token segment at degree 4
    (16q/1kv) plus a degree-1 tail (64q/4kv) filling 16,384 tokens. About 1.9 GB on the device; the q tiles of the long
    group (16 heads) still exceed L2, which is what makes this shape's backward pass DRAM-heavy."""
    short = lognormal_lengths(seed, 16384, 4096, 1.0, 64, 65536)
    return _mk("large_head_profile_case_16k", [16384] + short, [16] + [64] * len(short), [1] + [4] * len(short), seed,
               "one 16,384-token segment (16q/1kv) + degree-1 tail (64q/4kv) filling 16,384 tokens")


def ragged(seed: int = 11) -> Workload:
    """Lengths that are not multiples of 16 or of any tile, a 1-token and a zero-length segment, three runs."""
    lengths = [1, 17, 0, 127, 129, 255, 1000, 3, 384]
    hq = [8, 8, 8, 4, 4, 4, 16, 16, 16]
    hkv = [2, 2, 2, 1, 1, 1, 16, 16, 16]
    return _mk("ragged_tails", lengths, hq, hkv, seed, "tail tiles, MQA/GQA/MHA runs, empty segment")


def custom(lengths, hq, hkv, seed: int = 0, name: str = "custom", head_dim: int = HEAD_DIM) -> Workload:
    n = len(lengths)
    hq = [hq] * n if np.isscalar(hq) else hq
    hkv = [hkv] * n if np.isscalar(hkv) else hkv
    return _mk(name, lengths, hq, hkv, seed, head_dim=head_dim)


def make_tensors(w: Workload, seed: int | None = None, which=("q", "k", "v", "do")):
    """iid N(0,1) bf16 tensors (flat, packed layout) as CPU torch tensors, drawn in the order Q, K, V, dO."""
    import torch

    g = torch.Generator(device="cpu")
    g.manual_seed(int(w.seed if seed is None else seed))
    sizes = {"q": w.q_elems(), "k": w.kv_elems(), "v": w.kv_elems(), "do": w.q_elems()}
    out = {}
    for name in ("q", "k", "v", "do"):
        n = sizes[name]
        if name not in which:
            # keep the stream position independent of which tensors are requested
            chunk = 1 << 24
            left = n
            while left > 0:
                torch.randn(min(chunk, left), generator=g)
                left -= chunk
            continue
        t = torch.empty(n, dtype=torch.bfloat16)
        chunk = 1 << 24
        for a in range(0, n, chunk):
            b = min(n, a + chunk)
            t[a:b] = torch.randn(b - a, generator=g, dtype=torch.float32).to(torch.bfloat16)
        out[name] = t
    return out


def bf16_bits(t) -> np.ndarray:
    """View a CPU torch bf16 tensor as a numpy uint16 array of its bit patterns (no copy)."""
    import torch

    return t.view(torch.int16).numpy().view(np.uint16)
