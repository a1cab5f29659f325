"""Ulysses prologue / epilogue (paper Sec. 2.1 "Sequence Parallelism", Sec. 4.1.2): the exchange schedule on CPU ranks (gloo, world sizes 2 and
4, layout steps by a plain torch stand-in), and the library's CUDA layout kernels on one GPU against the same
stand-in, including an emulation of all ranks of a node in one process."""
import os
import socket

import numpy as np
import pytest
import torch


class TorchLayoutOps:
    """Plain torch indexing with the semantics of nsp_a2a_gather_heads / nsp_a2a_scatter_heads."""

    def gather(self, src, dst, tokens, heads, hpb, D, first, stream=None):
        src = src.reshape(tokens, heads, D)
        dst = dst.reshape(len(first), tokens, hpb, D)
        for p, f in enumerate(first):
            dst[p].copy_(src[:, f:f + hpb])

    def scatter(self, src, dst, tokens, heads, hpb, D, first, stream=None):
        src = src.reshape(len(first), tokens, hpb, D)
        dst = dst.reshape(tokens, heads, D)
        for h in range(heads):
            parts = [src[p][:, h - f] for p, f in enumerate(first) if f <= h < f + hpb]
            if len(parts) == 1:
                dst[:, h] = parts[0]
            elif parts:
                acc = torch.zeros_like(parts[0], dtype=torch.float32)
                for x in parts:  # block order, fp32
                    acc = acc + x.float()
                dst[:, h] = acc.to(dst.dtype)


    def gather_to(self, src, dst_tensors, dst_row, sample_off, tokens, heads, hpb, D, first, stream=None):
        src = src.reshape(tokens, heads, D)
        off = [int(x) for x in sample_off.tolist()]
        for p, f in enumerate(first):
            for j in range(len(off) - 1):
                r = int(dst_row[p][j])
                dst_tensors[p].reshape(-1, hpb, D)[r:r + off[j + 1] - off[j]] = src[off[j]:off[j + 1], f:f + hpb]


def _global(lengths, H, D, seed, dtype=torch.float32):
    g = torch.Generator().manual_seed(seed)
    return [torch.randn(L, H, D, generator=g).to(dtype) for L in lengths]


def _local(xs, d, r):
    return torch.cat([x[r * (x.shape[0] // d):(r + 1) * (x.shape[0] // d)] for x in xs])


def _worker(rank, world, port, hq, hkv):
    import torch.distributed as dist

    from paper_2609_22755_b200.ulysses import NodeLayout, UlyssesExchange

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        D = 16
        lengths = [8 * world, 0, 3 * world, 20 * world]
        lay = NodeLayout(lengths, world, rank, hq, hkv, D)
        ex = UlyssesExchange(lay, list(range(world)), ops=TorchLayoutOps())
        q = _global(lengths, hq, D, 1)
        kv = _global(lengths, hkv, D, 2)
        # prologue: complete sequences, this rank's heads
        got_q = ex.to_attention_layout(_local(q, world, rank), "q")
        want_q = torch.cat([x[:, lay.q_first[rank]:lay.q_first[rank] + lay.hq_loc] for x in q])
        assert torch.equal(got_q, want_q)
        got_k = ex.to_attention_layout(_local(kv, world, rank), "kv")
        want_k = torch.cat([x[:, lay.kv_first[rank]:lay.kv_first[rank] + lay.hkv_loc] for x in kv])
        assert torch.equal(got_k, want_k)
        # epilogue of a q-shaped tensor: the exact inverse
        back = ex.from_attention_layout(got_q, "q")
        assert torch.equal(back, _local(q, world, rank))
        # epilogue of dK: rank s contributes (s + 1) * its block; shared heads are summed over the sharing ranks
        part = got_k * float(rank + 1)
        got_dk = ex.from_attention_layout(part, "kv")
        want = torch.zeros(lay.t_loc, hkv, D)
        for s in range(world):
            f = lay.kv_first[s]
            blk = torch.cat([x[:, f:f + lay.hkv_loc] for x in kv]) * float(s + 1)  # what rank s holds, full length
            mine = torch.cat([blk[lay.full_off[j] + rank * lay.tok_loc[j]:lay.full_off[j] + (rank + 1) * lay.tok_loc[j]]
                              for j in range(len(lengths))])
            want[:, f:f + lay.hkv_loc] += mine
        assert torch.allclose(got_dk, want, rtol=0, atol=1e-5)
    finally:
        dist.destroy_process_group()


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


@pytest.mark.parametrize("world,hq,hkv", [(2, 8, 4), (2, 4, 1), (4, 8, 2), (4, 8, 8), (8, 32, 4), (8, 8, 2)])
def test_exchange_schedule_on_cpu_ranks(world, hq, hkv):
    import torch.multiprocessing as mp

    mp.spawn(_worker, args=(world, _free_port(), hq, hkv), nprocs=world, join=True)


@pytest.mark.parametrize("d,hq,hkv", [(2, 8, 4), (4, 8, 2), (8, 32, 4)])
def test_fused_prologue_rows_on_cpu(d, hq, hkv):
    """Where the fused send side puts every block: all ranks of a node in one process, the stores done by the plain
    torch stand-in; every rank's attention buffer must come out as the global slicing."""
    from paper_2609_22755_b200.ulysses import NodeLayout, UlyssesExchange

    D = 16
    lengths = [8 * d, 0, 3 * d, 20 * d]
    for kind, H, seed in (("q", hq, 1), ("kv", hkv, 2)):
        xs = _global(lengths, H, D, seed)
        lays = [NodeLayout(lengths, d, r, hq, hkv, D) for r in range(d)]
        _, h_loc, first = lays[0].heads(kind)
        bufs = [torch.full((lays[0].t_full, h_loc, D), float("nan")) for _ in range(d)]
        for r, lay in enumerate(lays):
            UlyssesExchange(lay, list(range(d)), ops=TorchLayoutOps()).store_to_attention_layouts(
                _local(xs, d, r).contiguous(), kind, bufs)
        for r in range(d):
            assert torch.equal(bufs[r], torch.cat([x[:, first[r]:first[r] + h_loc] for x in xs]))


def test_layout_rejects_bad_shapes():
    from paper_2609_22755_b200.ulysses import NodeLayout

    with pytest.raises(ValueError):
        NodeLayout([10], 4, 0, 8, 2)  # length not a multiple of the degree
    with pytest.raises(ValueError):
        NodeLayout([16], 4, 0, 6, 2)  # degree does not divide the query heads
    with pytest.raises(ValueError):
        NodeLayout([16], 4, 4, 8, 2)  # rank outside the group
    lay = NodeLayout([16, 32], 4, 1, 8, 2)
    assert lay.kv_first == [0, 0, 1, 1] and lay.hkv_loc == 1 and lay.q_first == [0, 2, 4, 6]
    assert lay.t_loc == 12 and lay.t_full == 48


@pytest.mark.gpu
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("d,hq,hkv", [(2, 8, 4), (4, 8, 2), (8, 32, 4)])
def test_cuda_layout_kernels_and_one_process_emulation(d, hq, hkv, dtype):
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2609_22755_b200.ulysses import CudaLayoutOps, NodeLayout

    D = 128
    dev = torch.device("cuda:0")
    lengths = [64 * d, 8 * d, 0, 1000 * d]
    q = [x.to(dev) for x in _global(lengths, hq, D, 3, dtype)]
    kv = [x.to(dev) for x in _global(lengths, hkv, D, 4, dtype)]
    cuda_ops, ref_ops = CudaLayoutOps(), TorchLayoutOps()
    lays = [NodeLayout(lengths, d, r, hq, hkv, D) for r in range(d)]
    sends = {}
    for kind, xs in (("q", q), ("kv", kv)):
        for r, lay in enumerate(lays):
            H, h_loc, first = lay.heads(kind)
            x_loc = _local(xs, d, r).contiguous()
            got = torch.empty((d, lay.t_loc, h_loc, D), dtype=dtype, device=dev)
            want = torch.empty_like(got)
            cuda_ops.gather(x_loc, got, lay.t_loc, H, h_loc, D, first)
            ref_ops.gather(x_loc, want, lay.t_loc, H, h_loc, D, first)
            assert torch.equal(got, want)
            sends[kind, r] = got
    # all ranks in one process: move the blocks the way the exchange does and compare with the global slicing
    for kind, xs in (("q", q), ("kv", kv)):
        for r, lay in enumerate(lays):
            H, h_loc, first = lay.heads(kind)
            full = torch.empty((lay.t_full, h_loc, D), dtype=dtype, device=dev)
            for s in range(d):
                for j in range(len(lengths)):
                    a = int(lay.full_off[j]) + s * lay.tok_loc[j]
                    full[a:a + lay.tok_loc[j]] = sends[kind, s][r, int(lay.loc_off[j]):int(lay.loc_off[j + 1])]
            assert torch.equal(full, torch.cat([x[:, first[r]:first[r] + h_loc] for x in xs]))
    # the fused send side: every "rank" stores its slices straight into the attention buffers of all ranks (all of
    # them local here: one GPU stands for the node); the buffers must equal the global slicing bit for bit
    from paper_2609_22755_b200.ulysses import UlyssesExchange

    for kind, xs in (("q", q), ("kv", kv)):
        H, h_loc, first = lays[0].heads(kind)
        bufs = [torch.full((lays[0].t_full, h_loc, D), float("nan"), dtype=dtype, device=dev) for _ in range(d)]
        for r, lay in enumerate(lays):
            UlyssesExchange(lay, list(range(d))).store_to_attention_layouts(_local(xs, d, r).contiguous(), kind, bufs)
        for r in range(d):
            assert torch.equal(bufs[r], torch.cat([x[:, first[r]:first[r] + h_loc] for x in xs]))
    # scatter: inverse for q; sums for shared KV heads
    for kind in ("q", "kv"):
        lay = lays[0]
        H, h_loc, first = lay.heads(kind)
        g = torch.Generator(device=dev).manual_seed(5)
        blocks = torch.randn((d, lay.t_loc, h_loc, D), device=dev, generator=g).to(dtype)
        got = torch.full((lay.t_loc, H, D), 7.0, dtype=dtype, device=dev)
        want = got.clone()
        cuda_ops.scatter(blocks, got, lay.t_loc, H, h_loc, D, first)
        ref_ops.scatter(blocks, want, lay.t_loc, H, h_loc, D, first)
        assert torch.equal(got, want)


@pytest.mark.gpu
def test_phase_streams_orders_the_phases_on_one_gpu():
    """Two-queue phase streaming with the exchange replaced by its layout step alone (one GPU, no peers): every
    node's result must equal what the three phases give when run one after the other on one stream."""
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2609_22755_b200 import binding as B
    from paper_2609_22755_b200 import workloads as W
    from paper_2609_22755_b200.ulysses import phase_streams

    dev = torch.device("cuda:0")
    D = 128
    nodes = [W.custom([2048, 512], 8, 2, seed=1), W.custom([4096], 4, 1, seed=2), W.custom([256] * 6, 16, 4, seed=3)]
    plans = [B.nsp_plan_tiles(w.cu_seqlens, w.hq, w.hkv, D) for w in nodes]
    host = [W.make_tensors(w, which=("q", "k", "v")) for w in nodes]
    staged = [{n: t.to(dev) for n, t in h.items() if n in ("q", "k", "v")} for h in host]

    def prologue(i):  # stands for the all-to-all: a head gather of the whole tensor into one block
        w, out = nodes[i], {}
        T = int(w.lengths.sum())
        for name, H in (("q", int(w.hq[0])), ("k", int(w.hkv[0])), ("v", int(w.hkv[0]))):
            dst = torch.empty_like(staged[i][name])
            B.nsp_a2a_gather_heads(staged[i][name], dst, T, H, H, D, [0], torch.cuda.current_stream())
            out[name] = dst
        return out

    def compute(i, x):
        w = nodes[i]
        o = torch.empty_like(x["q"])
        lse = torch.empty(w.lse_elems(), dtype=torch.float32, device=dev)
        B.nsp_attn_fwd(plans[i], x["q"], x["k"], x["v"], o, lse, w.softmax_scale, stream=torch.cuda.current_stream())
        return o

    def epilogue(i, o):
        w = nodes[i]
        out = torch.empty_like(o)
        B.nsp_a2a_scatter_heads(o, out, int(w.lengths.sum()), int(w.hq[0]), int(w.hq[0]), D, [0],
                                torch.cuda.current_stream())
        return out

    want = [epilogue(i, compute(i, prologue(i))) for i in range(len(nodes))]
    torch.cuda.synchronize()
    got = phase_streams(nodes, prologue, compute, epilogue)
    torch.cuda.synchronize()
    for g, w_ in zip(got, want):
        assert torch.equal(g, w_)
    assert all(B.nsp_device_status(p)[0] == 0 for p in plans)
