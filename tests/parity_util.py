"""Helpers for the GPU parity tests: run the CUDA path through the C ABI, run the oracle, compare.

Tolerances (benchmark definition): max-abs error 2e-2 and relative L2 error 1e-2 for O, dQ, dK, dV against the
fp64 oracle evaluated on the same bf16 input bytes. The graded gradient dtypes are dQ bf16, dK/dV fp32.
"""
from __future__ import annotations

import numpy as np

MAX_ABS_TOL = 2e-2
REL_L2_TOL = 1e-2
LSE_ABS_TOL = 2e-3


def errors(got: np.ndarray, want: np.ndarray):
    got = np.asarray(got, np.float64).ravel()
    want = np.asarray(want, np.float64).ravel()
    if want.size == 0:
        return 0.0, 0.0
    d = got - want
    max_abs = float(np.max(np.abs(d)))
    denom = float(np.sqrt((want * want).sum()))
    rel = float(np.sqrt((d * d).sum()) / denom) if denom > 0 else float(np.sqrt((d * d).sum()))
    return max_abs, rel


def check(name, got, want, max_abs_tol=MAX_ABS_TOL, rel_tol=REL_L2_TOL):
    assert np.all(np.isfinite(np.asarray(got, np.float64))), f"{name}: non-finite values in the GPU result"
    ma, rl = errors(got, want)
    assert ma <= max_abs_tol, f"{name}: max-abs error {ma:.4g} > {max_abs_tol}"
    assert rl <= rel_tol, f"{name}: relative L2 error {rl:.4g} > {rel_tol}"
    return ma, rl


class GpuRun:
    """Device buffers + one forward/backward through the C ABI for a workload."""

    def __init__(self, w, tensors=None, dq_dtype="bf16", dkv_dtype="f32", device="cuda:0", deterministic=False):
        import torch

        from paper_2609_22755_b200 import binding as B
        from paper_2609_22755_b200 import workloads as W

        self.torch, self.B, self.w = torch, B, w
        self.dev = torch.device(device)
        self.host = tensors if tensors is not None else W.make_tensors(w)
        self.q, self.k, self.v, self.do = (self.host[n].to(self.dev) for n in ("q", "k", "v", "do"))
        # deterministic: False, True (ordered additions) or "rounded" (terms rounded to a fixed quantum)
        flag = B.NSP_PLAN_ROUNDED_DQ if deterministic == "rounded" else B.NSP_PLAN_DETERMINISTIC_DQ
        opts = (128, 128, 1, flag) if deterministic else None
        self.plan = B.nsp_plan_tiles(w.cu_seqlens, w.hq, w.hkv, w.head_dim, opts=opts)
        assert self.plan.q_elems == w.q_elems() and self.plan.kv_elems == w.kv_elems()
        assert self.plan.lse_elems == w.lse_elems()
        # Every buffer the library writes sits between two 4 KiB guard bands filled with a byte pattern; results()
        # checks that the bands are untouched (a stand-in for a memory checker: an out-of-range store of a kernel
        # shows up as a failed test instead of silent corruption). Outputs start as NaN so that an element nobody
        # wrote is seen as well.
        self._guards = []
        tq = torch.float32 if dq_dtype == "f32" else torch.bfloat16
        tkv = torch.float32 if dkv_dtype == "f32" else torch.bfloat16
        self.o = self._guarded(w.q_elems(), torch.bfloat16)
        self.lse = self._guarded(w.lse_elems(), torch.float32)
        self.dq = self._guarded(w.q_elems(), tq)
        self.dk = self._guarded(w.kv_elems(), tkv)
        self.dv = self._guarded(w.kv_elems(), tkv)
        self.ws = self._guarded(max(self.plan.bwd_ws_bytes, 256), torch.uint8, fill=None)

    GUARD_BYTES = 4096
    GUARD_PATTERN = 0xA5

    def _guarded(self, n, dtype, fill=float("nan")):
        torch = self.torch
        size = torch.empty((), dtype=dtype).element_size()
        raw = torch.full((2 * self.GUARD_BYTES + n * size,), self.GUARD_PATTERN, dtype=torch.uint8, device=self.dev)
        body = raw[self.GUARD_BYTES:self.GUARD_BYTES + n * size].view(dtype)
        if fill is not None and n:
            body.fill_(fill)
        self._guards.append(raw)
        return body

    def check_guards(self):
        torch = self.torch
        for i, raw in enumerate(self._guards):
            lo, hi = raw[:self.GUARD_BYTES], raw[raw.numel() - self.GUARD_BYTES:]
            assert bool((lo == self.GUARD_PATTERN).all()) and bool((hi == self.GUARD_PATTERN).all()), \
                f"guard band of output buffer {i} was overwritten"

    def forward(self):
        self.B.nsp_attn_fwd(self.plan, self.q, self.k, self.v, self.o, self.lse, self.w.softmax_scale)

    def backward(self):
        self.B.nsp_attn_bwd(self.plan, self.q, self.k, self.v, self.o, self.do, self.lse, self.dq, self.dk, self.dv,
                            self.w.softmax_scale, self.ws)

    def status(self):
        return self.B.nsp_device_status(self.plan)

    def results(self):
        t = self.torch
        t.cuda.synchronize()
        self.check_guards()
        f = lambda x: x.float().cpu().numpy().astype(np.float64)
        return {"o": f(self.o), "lse": f(self.lse), "dq": f(self.dq), "dk": f(self.dk), "dv": f(self.dv)}


def oracle_full(w, host):
    import oracle
    from paper_2609_22755_b200 import workloads as W

    b = {n: W.bf16_bits(host[n]) for n in ("q", "k", "v", "do")}
    O, LSE = oracle.attn_fwd(b["q"], b["k"], b["v"], w.cu_seqlens, w.hq, w.hkv, w.head_dim, w.softmax_scale)
    dQ, dK, dV = oracle.attn_bwd(b["q"], b["k"], b["v"], b["do"], w.cu_seqlens, w.hq, w.hkv, w.head_dim,
                                 w.softmax_scale)
    return {"o": O, "lse": LSE, "dq": dQ, "dk": dK, "dv": dV}


def compare_full(w, res, ref, tag=""):
    out = {}
    for name in ("o", "dq", "dk", "dv"):
        out[name] = check(f"{w.name}{tag}:{name}", res[name], ref[name])
    if ref["lse"].size:
        d = float(np.max(np.abs(res["lse"] - ref["lse"])))
        assert d <= LSE_ABS_TOL, f"{w.name}{tag}: LSE max-abs error {d:.4g}"
        out["lse"] = (d, 0.0)
    return out
