"""Ulysses prologue / epilogue of one SP-tree node (paper Sec. 2.1; the communication phases of Sec. 4.1.2).

Before attention, every GPU of a degree-d node holds a 1/d token slice of each of the node's samples with all heads;
attention needs complete sequences with 1/d of the heads. The exchange is an all-to-all among the d GPUs. Here it is
issued as grouped point-to-point operations, one per (peer, sample), because that lets every received block land
directly where the attention kernels read it: the block a peer s sends for sample j is the token range
[s L_j / d, (s + 1) L_j / d) of that sample for this GPU's heads, which is a contiguous piece of the sample's
[L_j, H / d, D] segment in the packed token-major layout. Only the sending side needs a layout step (the head slice of
a token-major tensor is strided): ``nsp_a2a_gather_heads`` before the exchange, ``nsp_a2a_scatter_heads`` after the
reverse exchange (which also adds the partial dK / dV of a KV head that several GPUs of the node share).

The layout steps run in the library's CUDA kernels (``CudaLayoutOps``); the exchange goes through
``torch.distributed`` (NCCL between GPUs). ``phase_streams`` runs the communication of the next node on its own stream
while the current node computes (the paper's inter-level phase streaming in its simplest, two-queue form).
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


class CudaLayoutOps:
    """The library's layout kernels."""

    def gather(self, src, dst, tokens, heads, heads_per_block, head_dim, first_head, stream=None):
        from . import binding as B

        B.nsp_a2a_gather_heads(src, dst, tokens, heads, heads_per_block, head_dim, first_head, stream)

    def scatter(self, src, dst, tokens, heads, heads_per_block, head_dim, first_head, stream=None):
        from . import binding as B

        B.nsp_a2a_scatter_heads(src, dst, tokens, heads, heads_per_block, head_dim, first_head, stream)

    def gather_to(self, src, dst_tensors, dst_row, sample_off, tokens, heads, heads_per_block, head_dim, first_head,
                  stream=None):
        from . import binding as B

        B.nsp_a2a_gather_heads_to(src, dst_tensors, dst_row, sample_off, tokens, heads, heads_per_block, head_dim,
                                  first_head, stream)


@dataclass
class NodeLayout:
    """One SP-tree node as one of its GPUs sees it. lengths: full lengths of the node's samples (multiples of the
    degree); hq / hkv: heads of the whole model."""

    lengths: list
    degree: int
    rank: int  # position of this GPU inside the node's group
    hq: int
    hkv: int
    head_dim: int = 128

    def __post_init__(self):
        d = self.degree
        if d < 1 or not 0 <= self.rank < d:
            raise ValueError("rank must lie inside the group")
        if any(int(L) % d for L in self.lengths):
            raise ValueError("every sample length must be a multiple of the SP degree")
        if self.hq % d:
            raise ValueError("the SP degree must divide the number of query heads")
        if self.hkv % d and d % self.hkv:
            raise ValueError("the number of KV heads and the SP degree must divide one another")
        self.tok_loc = [int(L) // d for L in self.lengths]
        self.t_loc = int(sum(self.tok_loc))
        self.t_full = int(sum(int(L) for L in self.lengths))
        self.hq_loc = self.hq // d
        self.hkv_loc = max(1, self.hkv // d)
        self.q_first = [t * self.hq_loc for t in range(d)]
        self.kv_first = [(t * self.hkv) // d for t in range(d)]  # several peers share a head when hkv < d
        self.loc_off = np.concatenate([[0], np.cumsum(self.tok_loc)]).astype(np.int64)
        self.full_off = np.concatenate([[0], np.cumsum([int(L) for L in self.lengths])]).astype(np.int64)

    def heads(self, kind):
        """(heads of the whole tensor, heads per peer, first head per peer) for 'q' or 'kv' shaped tensors."""
        return (self.hq, self.hq_loc, self.q_first) if kind == "q" else (self.hkv, self.hkv_loc, self.kv_first)

    def workload_segments(self):
        """Lengths and local head counts of this node's segments in the attention layout."""
        return [int(L) for L in self.lengths], self.hq_loc, self.hkv_loc


class UlyssesExchange:
    """Prologue / epilogue of one node. group_ranks: the global ranks of the node's GPUs in group order."""

    def __init__(self, layout: NodeLayout, group_ranks, ops=None, group=None):
        self.lay = layout
        self.ranks = list(group_ranks)
        if len(self.ranks) != layout.degree:
            raise ValueError("group_ranks must list one global rank per GPU of the node")
        self.ops = ops if ops is not None else CudaLayoutOps()
        self.group = group

    def _exchange(self, send_of, recv_of):
        """One grouped exchange: send_of(peer, sample) / recv_of(peer, sample) return contiguous tensors."""
        import torch.distributed as dist

        lay = self.lay
        ops = []
        for p in range(lay.degree):
            for j in range(len(lay.lengths)):
                if lay.tok_loc[j] == 0:
                    continue
                if p == lay.rank:
                    recv_of(p, j).copy_(send_of(p, j))
                else:
                    ops.append(dist.P2POp(dist.isend, send_of(p, j), self.ranks[p], self.group))
                    ops.append(dist.P2POp(dist.irecv, recv_of(p, j), self.ranks[p], self.group))
        if ops:
            for req in dist.batch_isend_irecv(ops):
                req.wait()

    def to_attention_layout(self, x_loc, kind, out=None, stream=None):
        """x_loc [t_loc, H, D] (this GPU's token slices, all heads) -> [t_full, H / d, D]: complete sequences of the
        node's samples, this GPU's heads, packed sample after sample (what nsp_attn_fwd / nsp_attn_bwd read)."""
        import torch

        lay = self.lay
        H, h_loc, first = lay.heads(kind)
        D = lay.head_dim
        x_loc = x_loc.reshape(lay.t_loc, H, D)
        send = torch.empty((lay.degree, lay.t_loc, h_loc, D), dtype=x_loc.dtype, device=x_loc.device)
        self.ops.gather(x_loc, send, lay.t_loc, H, h_loc, D, first, stream)
        if out is None:
            out = torch.empty((lay.t_full, h_loc, D), dtype=x_loc.dtype, device=x_loc.device)
        out = out.reshape(lay.t_full, h_loc, D)

        def send_of(p, j):
            return send[p, lay.loc_off[j]:lay.loc_off[j + 1]]

        def recv_of(p, j):  # peer p holds the token range [p L_j / d, (p + 1) L_j / d) of sample j
            a = lay.full_off[j] + p * lay.tok_loc[j]
            return out[a:a + lay.tok_loc[j]]

        self._exchange(send_of, recv_of)
        return out

    def store_to_attention_layouts(self, x_loc, kind, peer_buffers, stream=None):
        """The prologue without a staging buffer and without a separate exchange: this GPU's token slices go, head block
        by head block, straight into the packed attention buffers of the node's GPUs. peer_buffers[p] is GPU p's
        [t_full, H / d, D] buffer as a tensor this process can write (its own for p == rank; a peer's memory mapped
        into this process otherwise, e.g. through CUDA IPC or a symmetric-memory allocation). One kernel of the library
        issues plain stores; the caller orders it against the readers (every GPU of the node runs this call, then the
        group synchronises, then attention runs)."""
        import torch

        lay = self.lay
        H, h_loc, first = lay.heads(kind)
        D = lay.head_dim
        x_loc = x_loc.reshape(lay.t_loc, H, D)
        if len(peer_buffers) != lay.degree:
            raise ValueError("one attention buffer per GPU of the node")
        # this GPU holds the token range [rank L_j / d, (rank + 1) L_j / d) of sample j, for every receiver alike
        rows = [[int(lay.full_off[j]) + lay.rank * lay.tok_loc[j] for j in range(len(lay.lengths))]] * lay.degree
        dst_row = torch.tensor(rows, dtype=torch.int64, device=x_loc.device)
        sample_off = torch.as_tensor(lay.loc_off, dtype=torch.int64).to(x_loc.device)
        self.ops.gather_to(x_loc, list(peer_buffers), dst_row, sample_off, lay.t_loc, H, h_loc, D, first, stream)

    def from_attention_layout(self, y_full, kind, out=None, stream=None):
        """The reverse: y_full [t_full, H / d, D] -> [t_loc, H, D]. Blocks that carry the same head (partial dK / dV of
        a KV head shared by several GPUs) are added in fp32."""
        import torch

        lay = self.lay
        H, h_loc, first = lay.heads(kind)
        D = lay.head_dim
        y_full = y_full.reshape(lay.t_full, h_loc, D)
        recv = torch.empty((lay.degree, lay.t_loc, h_loc, D), dtype=y_full.dtype, device=y_full.device)

        def send_of(p, j):
            a = lay.full_off[j] + p * lay.tok_loc[j]
            return y_full[a:a + lay.tok_loc[j]]

        def recv_of(p, j):
            return recv[p, lay.loc_off[j]:lay.loc_off[j + 1]]

        self._exchange(send_of, recv_of)
        if out is None:
            out = torch.empty((lay.t_loc, H, D), dtype=y_full.dtype, device=y_full.device)
        out = out.reshape(lay.t_loc, H, D)
        self.ops.scatter(recv, out, lay.t_loc, H, h_loc, D, first, stream)
        return out


def phase_streams(nodes, prologue, compute, epilogue):
    """Two-queue phase streaming over the nodes of a GPU's chain: the prologue of node i + 1 and the epilogue of node
    i - 1 run on a communication stream while node i computes. prologue(i) / compute(i, inputs) / epilogue(i, outputs)
    are callables; each is issued under the stream it belongs to and ordered with CUDA events. Returns the list of
    epilogue results. Tensors a phase allocates cross streams: the caller keeps them alive until the returned results
    have been consumed (as the lists here do). Without CUDA (CPU tensors) the phases simply run in order."""
    import torch

    if not torch.cuda.is_available():
        return [epilogue(i, compute(i, prologue(i))) for i in range(len(nodes))]
    comp = torch.cuda.current_stream()
    comm = torch.cuda.Stream()
    results = [None] * len(nodes)
    inputs, in_ready = [None] * len(nodes), [None] * len(nodes)
    comm.wait_stream(comp)

    def issue_prologue(i):
        with torch.cuda.stream(comm):
            inputs[i] = prologue(i)
            in_ready[i] = torch.cuda.Event()
            in_ready[i].record(comm)

    if nodes:
        issue_prologue(0)
    for i in range(len(nodes)):
        if i + 1 < len(nodes):
            issue_prologue(i + 1)  # overlaps compute(i)
        comp.wait_event(in_ready[i])
        outputs = compute(i, inputs[i])
        done = torch.cuda.Event()
        done.record(comp)
        with torch.cuda.stream(comm):
            comm.wait_event(done)
            results[i] = epilogue(i, outputs)  # overlaps compute(i + 1)
    comp.wait_stream(comm)
    return results
