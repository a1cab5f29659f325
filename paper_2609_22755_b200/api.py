"""User-facing wrapper: one object per packed batch that owns the plan and the device buffers and runs the
forward + backward of the local attention compute phase through the C ABI.

Only marshalling lives here. ``step_device`` runs on tensors already resident on the GPU; ``step_host`` is the
end-to-end call: it copies Q, K, V, dO from (pinned) host tensors, runs forward and backward, and copies
O, LSE, dQ, dK, dV back to host tensors; the copies run on a second stream under the kernels where the data
dependencies allow.
"""
from __future__ import annotations

from . import binding as B


class NspAttention:
    def __init__(self, workload, device="cuda:0", dq_dtype="bf16", dkv_dtype="f32", stream=None):
        import torch

        self.torch = torch
        self.w = workload
        self.dev = torch.device(device)
        torch.cuda.set_device(self.dev)
        self.stream = stream
        self.plan = B.nsp_plan_tiles(workload.cu_seqlens, workload.hq, workload.hkv, workload.head_dim, stream=stream)
        qe, kve, le = self.plan.q_elems, self.plan.kv_elems, self.plan.lse_elems
        bf, f32 = torch.bfloat16, torch.float32
        mk = lambda n, dt: torch.empty(n, dtype=dt, device=self.dev)
        self.q, self.k, self.v, self.do = mk(qe, bf), mk(kve, bf), mk(kve, bf), mk(qe, bf)
        self.o, self.lse = mk(qe, bf), mk(le, f32)
        self.dq = mk(qe, f32 if dq_dtype == "f32" else bf)
        self.dk = mk(kve, f32 if dkv_dtype == "f32" else bf)
        self.dv = mk(kve, f32 if dkv_dtype == "f32" else bf)
        self.ws = torch.empty(max(self.plan.bwd_ws_bytes, 256), dtype=torch.uint8, device=self.dev)
        self.scale = workload.softmax_scale

    # ---- data movement
    def load(self, host):
        """Copy Q, K, V, dO from host tensors (dict with keys q, k, v, do)."""
        for name, dst in (("q", self.q), ("k", self.k), ("v", self.v), ("do", self.do)):
            dst.copy_(host[name], non_blocking=True)
        return sum(host[n].numel() * host[n].element_size() for n in ("q", "k", "v", "do"))

    def store(self, host_out):
        """Copy O, LSE, dQ, dK, dV to host tensors (dict with keys o, lse, dq, dk, dv)."""
        n = 0
        for name, src in (("o", self.o), ("lse", self.lse), ("dq", self.dq), ("dk", self.dk), ("dv", self.dv)):
            host_out[name].copy_(src, non_blocking=True)
            n += src.numel() * src.element_size()
        return n

    def alloc_host_outputs(self):
        t = self.torch
        return {name: t.empty(src.shape, dtype=src.dtype, pin_memory=True)
                for name, src in (("o", self.o), ("lse", self.lse), ("dq", self.dq), ("dk", self.dk), ("dv", self.dv))}

    # ---- compute
    def forward(self):
        B.nsp_attn_fwd(self.plan, self.q, self.k, self.v, self.o, self.lse, self.scale, stream=self.stream)

    def backward(self, recompute=None):
        """recompute: optional uint8 flags per segment (see nsp_recompute_mark): O and LSE of a flagged segment are
        not read, the backward pass recomputes what it needs of them."""
        if recompute is None:
            B.nsp_attn_bwd(self.plan, self.q, self.k, self.v, self.o, self.do, self.lse, self.dq, self.dk, self.dv,
                           self.scale, self.ws, stream=self.stream)
            return
        need = B.nsp_plan_recompute_ws_bytes(self.plan)
        if self.ws.numel() < need:
            self.ws = self.torch.empty(need, dtype=self.torch.uint8, device=self.dev)
        B.nsp_attn_bwd_recompute(self.plan, recompute, self.q, self.k, self.v, self.o, self.do, self.lse, self.dq,
                                 self.dk, self.dv, self.scale, self.ws, stream=self.stream)

    def step_device(self):
        self.forward()
        self.backward()

    def step_host(self, host_in, host_out):
        """End to end: host tensors in, host tensors out. The copies run on a second stream, ordered with events, so
        that dO travels to the device while the forward pass runs and O / LSE travel back while the backward pass
        runs; what stays exposed is the copy of Q, K, V before the forward and of dQ, dK, dV after the backward.
        Returns (host-to-device bytes, device-to-host bytes). The call returns without waiting for the device."""
        torch = self.torch
        comp = torch.cuda.current_stream() if self.stream is None else self.stream
        if getattr(self, "_copy_stream", None) is None:
            self._copy_stream = torch.cuda.Stream(device=self.dev)
        cp = self._copy_stream
        size = lambda t: t.numel() * t.element_size()
        cp.wait_stream(comp)  # the buffers of the previous step are free
        with torch.cuda.stream(cp):
            for name, dst in (("q", self.q), ("k", self.k), ("v", self.v)):
                dst.copy_(host_in[name], non_blocking=True)
            qkv_in = torch.cuda.Event()
            qkv_in.record(cp)
            self.do.copy_(host_in["do"], non_blocking=True)
            do_in = torch.cuda.Event()
            do_in.record(cp)
        comp.wait_event(qkv_in)
        self.forward()
        fwd_done = torch.cuda.Event()
        fwd_done.record(comp)
        with torch.cuda.stream(cp):
            cp.wait_event(fwd_done)
            host_out["o"].copy_(self.o, non_blocking=True)
            host_out["lse"].copy_(self.lse, non_blocking=True)
        comp.wait_event(do_in)
        self.backward()
        bwd_done = torch.cuda.Event()
        bwd_done.record(comp)
        with torch.cuda.stream(cp):
            cp.wait_event(bwd_done)
            for name, src in (("dq", self.dq), ("dk", self.dk), ("dv", self.dv)):
                host_out[name].copy_(src, non_blocking=True)
        comp.wait_stream(cp)  # the step is complete on the caller's stream once the last copy is
        h2d = sum(size(host_in[n]) for n in ("q", "k", "v", "do"))
        d2h = sum(size(t) for t in (self.o, self.lse, self.dq, self.dk, self.dv))
        return h2d, d2h

    def status(self):
        return B.nsp_device_status(self.plan)
