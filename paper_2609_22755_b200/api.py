"""User-facing wrapper: one object per packed batch that owns the plan and the device buffers and runs the
forward + backward of the local attention compute phase through the C ABI.

Only marshalling lives here. ``step_device`` runs on tensors already resident on the GPU; ``step_host`` is the
end-to-end call (nsp_attn_step_host): Q, K, V, dO come from (pinned) host tensors and O, LSE, dQ, dK, dV go back to
host tensors; the library makes the copies on a second stream under the kernels where the data dependencies allow.
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
        """End to end: host tensors in (dict with q, k, v, do), host tensors out (dict with o, lse, dq, dk, dv), through
        the library's host-buffer entry point nsp_attn_step_host: the copies run on the plan's second stream, so that
        dO travels to the device while the forward pass runs and O / LSE travel back while the backward pass runs.
        The device copies live in a workspace of this object's own (not in the tensors step_device uses).
        Returns (host-to-device bytes, device-to-host bytes). The call returns without waiting for the device."""
        if getattr(self, "_host_ws", None) is None:
            dq_dt = B.NSP_F32 if host_out["dq"].dtype == self.torch.float32 else B.NSP_BF16
            dkv_dt = B.NSP_F32 if host_out["dk"].dtype == self.torch.float32 else B.NSP_BF16
            need = B.nsp_plan_step_host_ws_bytes(self.plan, dq_dt, dkv_dt)
            self._host_ws = self.torch.empty(max(need, 256), dtype=self.torch.uint8, device=self.dev)
        return B.nsp_attn_step_host(self.plan, host_in["q"], host_in["k"], host_in["v"], host_in["do"], host_out["o"],
                                    host_out["lse"], host_out["dq"], host_out["dk"], host_out["dv"], self.scale,
                                    self._host_ws, stream=self.stream)

    def status(self):
        return B.nsp_device_status(self.plan)
