"""ctypes binding of ``libnsp.so``: the same entry points as ``include/nsp.h``, argument marshalling only.

Every step of the path runs inside the CUDA library; torch is used here for device memory and streams. There is
no fallback: if the library has not been built (``python -m paper_2609_22755_b200.build``) importing the symbols
raises, and on a machine without a B200 the compute calls return ``NSP_ERR_CUDA`` / ``NSP_ERR_UNSUPPORTED``.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import numpy as np

NSP_OK = 0
NSP_ERR_INVALID_ARG = 1
NSP_ERR_UNSUPPORTED = 2
NSP_ERR_ALLOC = 3
NSP_ERR_CUDA = 4
NSP_ERR_DEVICE_TIMEOUT = 5
NSP_ERR_WORKSPACE = 6
NSP_ERR_DEVICE_ASSERT = 7
NSP_ERR_INFEASIBLE = 8
NSP_BF16 = 0
NSP_F32 = 1
NSP_MAX_RUNS = 32
NSP_PLAN_DETERMINISTIC_DQ = 1
NSP_PLAN_ROUNDED_DQ = 2

EXPORTS = [
    "nsp_plan_tiles", "nsp_plan_sizes", "nsp_plan_get", "nsp_attn_fwd", "nsp_attn_bwd", "nsp_device_status",
    "nsp_launch_count", "nsp_plan_destroy", "nsp_status_string", "nsp_plan_set_profiling", "nsp_plan_kernel_ms",
    "nsp_attn_bwd_static", "nsp_recompute_mark", "nsp_plan_recompute_ws_bytes", "nsp_attn_bwd_recompute",
    "nsp_cost_table", "nsp_route_sp_tree", "nsp_a2a_gather_heads", "nsp_a2a_scatter_heads",
    "nsp_selftest_wait_timeout", "nsp_a2a_gather_heads_to", "nsp_plan_set_wait_limit",
    "nsp_plan_step_host_ws_bytes", "nsp_attn_step_host",
]
CHECKED_EXPORTS = ["nsp_checked_withhold_load"]  # libnsp_checked.so only
NSP_COST_BUCKETS = 16
NSP_STATIC_WS_BYTES = 32 * 1024 * 1024
KERNEL_FWD, KERNEL_BWD_PRE, KERNEL_BWD_MAIN, KERNEL_BWD_POST, KERNEL_BWD_FIRST, KERNEL_FWD_FIRST = 0, 1, 2, 3, 4, 5

import os

# NSP_LIBRARY names another build of the same library (for instance the checked build, libnsp_checked.so, whose
# kernels verify every index they compute); the default is the library built next to this file.
LIB_PATH = Path(os.environ.get("NSP_LIBRARY", Path(__file__).resolve().parent / "libnsp.so"))
_lib = None


class NspError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        super().__init__(f"{what}: {status_string(code)} (code {code})")


class PlanOpts(ctypes.Structure):
    _fields_ = [("bm", ctypes.c_int32), ("bn", ctypes.c_int32), ("order_version", ctypes.c_int32),
                ("flags", ctypes.c_int32)]


def lib() -> ctypes.CDLL:
    """Load the CUDA library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not LIB_PATH.exists():
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2609_22755_b200.build` "
                              "(there is no CPU fallback)")
        L = ctypes.CDLL(str(LIB_PATH))
        vp, i32p, i64p = ctypes.c_void_p, ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_int64)
        L.nsp_plan_tiles.argtypes = [vp, vp, vp, ctypes.c_int32, ctypes.c_int32, vp, vp, ctypes.POINTER(vp)]
        L.nsp_plan_tiles.restype = ctypes.c_int
        L.nsp_plan_sizes.argtypes = [vp, i64p, i64p, i64p, ctypes.POINTER(ctypes.c_size_t), ctypes.POINTER(ctypes.c_size_t)]
        L.nsp_plan_sizes.restype = ctypes.c_int
        L.nsp_plan_get.argtypes = [vp, ctypes.c_int, vp, ctypes.c_int64, i64p]
        L.nsp_plan_get.restype = ctypes.c_int
        L.nsp_attn_fwd.argtypes = [vp, vp, vp, vp, vp, vp, ctypes.c_float, vp, ctypes.c_size_t, vp]
        L.nsp_attn_fwd.restype = ctypes.c_int
        L.nsp_attn_bwd.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, ctypes.c_int, ctypes.c_int, ctypes.c_float,
                                   vp, ctypes.c_size_t, vp]
        L.nsp_attn_bwd.restype = ctypes.c_int
        L.nsp_attn_bwd_static.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, ctypes.c_int, ctypes.c_int,
                                          ctypes.c_float, vp]
        L.nsp_attn_bwd_static.restype = ctypes.c_int
        L.nsp_recompute_mark.argtypes = [vp, vp, vp, ctypes.c_int32, ctypes.c_int32, ctypes.c_int64, vp, i64p]
        L.nsp_recompute_mark.restype = ctypes.c_int
        L.nsp_plan_recompute_ws_bytes.argtypes = [vp, ctypes.POINTER(ctypes.c_size_t)]
        L.nsp_plan_recompute_ws_bytes.restype = ctypes.c_int
        L.nsp_attn_bwd_recompute.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, ctypes.c_int, ctypes.c_int,
                                             ctypes.c_float, vp, ctypes.c_size_t, vp]
        L.nsp_attn_bwd_recompute.restype = ctypes.c_int
        L.nsp_cost_table.argtypes = [vp, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
                                     vp, vp, ctypes.c_double, vp]
        L.nsp_cost_table.restype = ctypes.c_int
        L.nsp_route_sp_tree.argtypes = [vp, vp, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
                                        ctypes.c_int64, ctypes.c_int32, vp, vp, vp, vp, i32p]
        L.nsp_route_sp_tree.restype = ctypes.c_int
        for f in (L.nsp_a2a_gather_heads, L.nsp_a2a_scatter_heads):
            f.argtypes = [vp, vp, ctypes.c_int64, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
                          ctypes.c_int32, vp, vp]
            f.restype = ctypes.c_int
        L.nsp_a2a_gather_heads_to.argtypes = [vp, vp, vp, vp, ctypes.c_int32, ctypes.c_int64, ctypes.c_int32, ctypes.c_int32,
                                              ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, vp, vp]
        L.nsp_a2a_gather_heads_to.restype = ctypes.c_int
        L.nsp_plan_step_host_ws_bytes.argtypes = [vp, ctypes.c_int, ctypes.c_int, ctypes.POINTER(ctypes.c_size_t)]
        L.nsp_plan_step_host_ws_bytes.restype = ctypes.c_int
        L.nsp_attn_step_host.argtypes = [vp] * 10 + [ctypes.c_int, ctypes.c_int, ctypes.c_float, vp, ctypes.c_size_t, vp]
        L.nsp_attn_step_host.restype = ctypes.c_int
        L.nsp_plan_set_wait_limit.argtypes = [vp, ctypes.c_int64]
        L.nsp_plan_set_wait_limit.restype = ctypes.c_int
        if hasattr(L, "nsp_checked_withhold_load"):
            L.nsp_checked_withhold_load.argtypes = [vp, ctypes.c_int]
            L.nsp_checked_withhold_load.restype = ctypes.c_int
        L.nsp_selftest_wait_timeout.argtypes = [vp, ctypes.c_int64, vp]
        L.nsp_selftest_wait_timeout.restype = ctypes.c_int
        L.nsp_device_status.argtypes = [vp, i32p]
        L.nsp_device_status.restype = ctypes.c_int
        L.nsp_launch_count.argtypes = []
        L.nsp_launch_count.restype = ctypes.c_int64
        L.nsp_plan_destroy.argtypes = [vp]
        L.nsp_plan_destroy.restype = ctypes.c_int
        L.nsp_plan_set_profiling.argtypes = [vp, ctypes.c_int]
        L.nsp_plan_set_profiling.restype = ctypes.c_int
        L.nsp_plan_kernel_ms.argtypes = [vp, ctypes.c_int, ctypes.POINTER(ctypes.c_float)]
        L.nsp_plan_kernel_ms.restype = ctypes.c_int
        L.nsp_status_string.argtypes = [ctypes.c_int]
        L.nsp_status_string.restype = ctypes.c_char_p
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().nsp_status_string(int(code)).decode()


def launch_count() -> int:
    return int(lib().nsp_launch_count())


def _i32(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _ptr(t):
    """Address of a torch tensor / numpy array (host metadata only) / int / None. Tensor arguments of the compute
    calls are validated by _check_tensors before they get here."""
    if t is None:
        return None
    if isinstance(t, int):
        return ctypes.c_void_p(t)
    if isinstance(t, np.ndarray):
        return t.ctypes.data_as(ctypes.c_void_p)
    return ctypes.c_void_p(t.data_ptr())


def _check_tensors(what, plan, specs):
    """Refuse buffers the kernels would read or write out of bounds: every tensor must be a contiguous CUDA tensor
    of the stated dtype with at least the plan's element count. specs: (name, tensor, allowed dtypes, min elements).
    Sizes of zero need no buffer at all."""
    import torch

    for name, t, dtypes, need in specs:
        if need == 0:
            continue
        if not isinstance(t, torch.Tensor) or not t.is_cuda or not t.is_contiguous():
            raise NspError(NSP_ERR_INVALID_ARG, f"{what}: {name} must be a contiguous CUDA tensor")
        if t.dtype not in dtypes:
            raise NspError(NSP_ERR_INVALID_ARG, f"{what}: {name} has dtype {t.dtype}")
        if t.numel() < need:
            raise NspError(NSP_ERR_INVALID_ARG, f"{what}: {name} holds {t.numel()} elements, the plan needs {need}")
        if t.device.index != torch.cuda.current_device():
            raise NspError(NSP_ERR_INVALID_ARG, f"{what}: {name} is on {t.device}, not on the current device")


def _fwd_specs(plan, q, k, v, o, lse):
    import torch

    bf, f32 = (torch.bfloat16,), (torch.float32,)
    return [("q", q, bf, plan.q_elems), ("k", k, bf, plan.kv_elems), ("v", v, bf, plan.kv_elems),
            ("o", o, bf, plan.q_elems), ("lse", lse, f32, plan.lse_elems)]


def _bwd_specs(plan, q, k, v, o, d_o, lse, dq, dk, dv, dq_dtype, dkv_dtype):
    import torch

    bf, f32 = (torch.bfloat16,), (torch.float32,)
    return _fwd_specs(plan, q, k, v, o, lse) + [
        ("d_o", d_o, bf, plan.q_elems), ("dq", dq, f32 if dq_dtype == NSP_F32 else bf, plan.q_elems),
        ("dk", dk, f32 if dkv_dtype == NSP_F32 else bf, plan.kv_elems),
        ("dv", dv, f32 if dkv_dtype == NSP_F32 else bf, plan.kv_elems)]


def _check_ws(what, ws):
    import torch

    if ws is not None and (not isinstance(ws, torch.Tensor) or not ws.is_cuda or not ws.is_contiguous()):
        raise NspError(NSP_ERR_WORKSPACE, f"{what}: the workspace must be a contiguous CUDA tensor")


def _stream_ptr(stream):
    if stream is None:
        import torch

        stream = torch.cuda.current_stream()
    if isinstance(stream, int):
        return ctypes.c_void_p(stream)
    return ctypes.c_void_p(stream.cuda_stream)


class Plan:
    """Owner of an ``nsp_plan_t*``."""

    def __init__(self, handle, n_seg):
        self.handle = handle
        self.n_seg = n_seg
        q, kv, l = ctypes.c_int64(), ctypes.c_int64(), ctypes.c_int64()
        fw, bw = ctypes.c_size_t(), ctypes.c_size_t()
        rc = lib().nsp_plan_sizes(handle, ctypes.byref(q), ctypes.byref(kv), ctypes.byref(l), ctypes.byref(fw),
                                  ctypes.byref(bw))
        if rc != NSP_OK:
            raise NspError(rc, "nsp_plan_sizes")
        self.q_elems, self.kv_elems, self.lse_elems = q.value, kv.value, l.value
        self.fwd_ws_bytes, self.bwd_ws_bytes = fw.value, bw.value

    def destroy(self):
        if self.handle:
            lib().nsp_plan_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def nsp_plan_tiles(cu_seqlens, hq, hkv, head_dim=128, opts=None, stream=None) -> Plan:
    cu, hq_, hkv_ = _i32(cu_seqlens), _i32(hq), _i32(hkv)
    n_seg = len(hq_)
    if len(cu) != n_seg + 1 or len(hkv_) != n_seg:
        raise NspError(NSP_ERR_INVALID_ARG, "nsp_plan_tiles(argument shapes)")
    o = None
    if opts is not None:
        o = PlanOpts(*opts)
    handle = ctypes.c_void_p()
    rc = lib().nsp_plan_tiles(_ptr(cu), _ptr(hq_), _ptr(hkv_), n_seg, head_dim, ctypes.byref(o) if o else None,
                              _stream_ptr(stream), ctypes.byref(handle))
    if rc != NSP_OK:
        raise NspError(rc, "nsp_plan_tiles")
    return Plan(handle, n_seg)


def nsp_plan_get(plan: Plan, pass_: int) -> np.ndarray:
    """The device work list as an int32 array [n_items, 4] = (seg, head, tile, cost)."""
    n = ctypes.c_int64()
    rc = lib().nsp_plan_get(plan.handle, pass_, None, 0, ctypes.byref(n))
    if rc != NSP_OK:
        raise NspError(rc, "nsp_plan_get")
    out = np.zeros((max(n.value, 1), 4), np.int32)
    rc = lib().nsp_plan_get(plan.handle, pass_, _ptr(out), n.value, ctypes.byref(n))
    if rc != NSP_OK:
        raise NspError(rc, "nsp_plan_get")
    return out[: n.value]


def nsp_attn_fwd(plan: Plan, q, k, v, o, lse, softmax_scale, ws=None, stream=None):
    _check_tensors("nsp_attn_fwd", plan, _fwd_specs(plan, q, k, v, o, lse))
    _check_ws("nsp_attn_fwd", ws)
    ws_bytes = 0 if ws is None else ws.numel() * ws.element_size()
    rc = lib().nsp_attn_fwd(plan.handle, _ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), float(softmax_scale), _ptr(ws),
                            ws_bytes, _stream_ptr(stream))
    if rc != NSP_OK:
        raise NspError(rc, "nsp_attn_fwd")


def nsp_attn_bwd(plan: Plan, q, k, v, o, d_o, lse, dq, dk, dv, softmax_scale, ws, dq_dtype=None, dkv_dtype=None,
                 stream=None):
    import torch

    if dq_dtype is None:
        dq_dtype = NSP_F32 if dq.dtype == torch.float32 else NSP_BF16
    if dkv_dtype is None:
        dkv_dtype = NSP_F32 if dk.dtype == torch.float32 else NSP_BF16
    if dq_dtype not in (NSP_BF16, NSP_F32) or dkv_dtype not in (NSP_BF16, NSP_F32):
        raise NspError(NSP_ERR_INVALID_ARG, "nsp_attn_bwd: gradient dtype")
    _check_tensors("nsp_attn_bwd", plan, _bwd_specs(plan, q, k, v, o, d_o, lse, dq, dk, dv, dq_dtype, dkv_dtype))
    _check_ws("nsp_attn_bwd", ws)
    ws_bytes = 0 if ws is None else ws.numel() * ws.element_size()
    rc = lib().nsp_attn_bwd(plan.handle, _ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(d_o), _ptr(lse), _ptr(dq), _ptr(dk),
                            _ptr(dv), dq_dtype, dkv_dtype, float(softmax_scale), _ptr(ws), ws_bytes,
                            _stream_ptr(stream))
    if rc != NSP_OK:
        raise NspError(rc, "nsp_attn_bwd")


def nsp_plan_step_host_ws_bytes(plan: Plan, dq_dtype=NSP_BF16, dkv_dtype=NSP_F32) -> int:
    n = ctypes.c_size_t()
    rc = lib().nsp_plan_step_host_ws_bytes(plan.handle, int(dq_dtype), int(dkv_dtype), ctypes.byref(n))
    if rc != NSP_OK:
        raise NspError(rc, "nsp_plan_step_host_ws_bytes")
    return int(n.value)


def nsp_attn_step_host(plan: Plan, h_q, h_k, h_v, h_do, h_o, h_lse, h_dq, h_dk, h_dv, softmax_scale, dev_ws, stream=None):
    """Forward + backward with host tensors in and out (CPU torch tensors, pinned for asynchronous copies); dev_ws is
    a CUDA uint8 tensor of at least nsp_plan_step_host_ws_bytes. Returns (host-to-device, device-to-host) bytes."""
    import torch

    bf, f32 = (torch.bfloat16,), (torch.float32,)
    dq_dtype = NSP_F32 if h_dq.dtype == torch.float32 else NSP_BF16
    dkv_dtype = NSP_F32 if h_dk.dtype == torch.float32 else NSP_BF16
    specs = [("h_q", h_q, bf, plan.q_elems), ("h_k", h_k, bf, plan.kv_elems), ("h_v", h_v, bf, plan.kv_elems),
             ("h_do", h_do, bf, plan.q_elems), ("h_o", h_o, bf, plan.q_elems), ("h_lse", h_lse, f32, plan.lse_elems),
             ("h_dq", h_dq, f32 + bf, plan.q_elems), ("h_dk", h_dk, f32 + bf, plan.kv_elems),
             ("h_dv", h_dv, (h_dk.dtype,), plan.kv_elems)]
    for name, t, dtypes, need in specs:
        if need == 0:
            continue
        if not isinstance(t, torch.Tensor) or t.is_cuda or not t.is_contiguous() or t.dtype not in dtypes or t.numel() < need:
            raise NspError(NSP_ERR_INVALID_ARG, f"nsp_attn_step_host: {name} must be a contiguous host tensor of "
                                                f"{need} elements of {dtypes}")
    _check_ws("nsp_attn_step_host", dev_ws)
    ws_bytes = 0 if dev_ws is None else dev_ws.numel() * dev_ws.element_size()
    rc = lib().nsp_attn_step_host(plan.handle, _ptr(h_q), _ptr(h_k), _ptr(h_v), _ptr(h_do), _ptr(h_o), _ptr(h_lse),
                                  _ptr(h_dq), _ptr(h_dk), _ptr(h_dv), dq_dtype, dkv_dtype, float(softmax_scale),
                                  _ptr(dev_ws), ws_bytes, _stream_ptr(stream))
    if rc != NSP_OK:
        raise NspError(rc, "nsp_attn_step_host")
    size = lambda t: t.numel() * t.element_size()
    return (sum(size(t) for t in (h_q, h_k, h_v, h_do)), sum(size(t) for t in (h_o, h_lse, h_dq, h_dk, h_dv)))


def nsp_recompute_mark(cu_seqlens, hq, level, budget_bytes: int, head_dim: int = 128):
    """Save / recompute marking of a shard's segments under an activation budget (host only); returns
    (flags uint8 [n_seg], bytes of the saved segments)."""
    import numpy as np

    cu = np.ascontiguousarray(cu_seqlens, dtype=np.int32)
    hq = np.ascontiguousarray(hq, dtype=np.int32)
    level = np.ascontiguousarray(level, dtype=np.int32)
    n = len(hq)
    if cu.shape != (n + 1,) or level.shape != (n,):
        raise ValueError("cu_seqlens needs n_seg + 1 entries, hq and level n_seg")
    flags = np.zeros(max(n, 1), dtype=np.uint8)
    saved = ctypes.c_int64()
    vp = ctypes.c_void_p
    rc = lib().nsp_recompute_mark(cu.ctypes.data_as(vp), hq.ctypes.data_as(vp), level.ctypes.data_as(vp), n,
                                  int(head_dim), int(budget_bytes), flags.ctypes.data_as(vp), ctypes.byref(saved))
    if rc != NSP_OK:
        raise NspError(rc, "nsp_recompute_mark")
    return flags[:n], int(saved.value)


def nsp_cost_table(lengths, n_levels, hq, hkv, head_dim, tcomp_ns, link_gbs, other_ns_per_token):
    """Cost table [n_samples, n_levels] (int64 ns per covered GPU) from profiled coefficients (host only)."""
    import numpy as np

    lengths = np.ascontiguousarray(lengths, dtype=np.int32)
    tcomp = np.ascontiguousarray(tcomp_ns, dtype=np.float64)
    link = np.ascontiguousarray(link_gbs, dtype=np.float64)
    if tcomp.shape != (n_levels, NSP_COST_BUCKETS) or link.shape != (n_levels,):
        raise ValueError("tcomp_ns must be [n_levels, NSP_COST_BUCKETS], link_gbs [n_levels]")
    out = np.zeros((len(lengths), n_levels), dtype=np.int64)
    vp = ctypes.c_void_p
    rc = lib().nsp_cost_table(lengths.ctypes.data_as(vp), len(lengths), int(n_levels), int(hq), int(hkv), int(head_dim),
                              tcomp.ctypes.data_as(vp), link.ctypes.data_as(vp), float(other_ns_per_token),
                              out.ctypes.data_as(vp))
    if rc != NSP_OK:
        raise NspError(rc, "nsp_cost_table")
    return out


def nsp_route_sp_tree(lengths, cost, n_levels, prefix_k, beam_w, b_tok, monotone=False):
    """Algorithm 1 (host only). Returns (level[n], index[n], load[P], tok[P] in 1/P tokens, feasible) or raises
    NspError(NSP_ERR_INFEASIBLE)."""
    import numpy as np

    lengths = np.ascontiguousarray(lengths, dtype=np.int32)
    cost = np.ascontiguousarray(cost, dtype=np.int64)
    n = len(lengths)
    if cost.shape != (n, n_levels):
        raise ValueError("cost must be [n_samples, n_levels]")
    P = 1 << (n_levels - 1)
    level = np.zeros(max(n, 1), np.int32)
    index = np.zeros(max(n, 1), np.int32)
    load = np.zeros(P, np.int64)
    tok = np.zeros(P, np.int64)
    feas = ctypes.c_int32()
    vp = ctypes.c_void_p
    rc = lib().nsp_route_sp_tree(lengths.ctypes.data_as(vp), cost.ctypes.data_as(vp), n, int(n_levels), int(prefix_k),
                                 int(beam_w), int(b_tok), int(bool(monotone)), level.ctypes.data_as(vp),
                                 index.ctypes.data_as(vp), load.ctypes.data_as(vp), tok.ctypes.data_as(vp),
                                 ctypes.byref(feas))
    if rc != NSP_OK:
        raise NspError(rc, "nsp_route_sp_tree")
    return level[:n], index[:n], load, tok, bool(feas.value)


def _a2a(fn_name, src, dst, tokens, heads, heads_per_block, head_dim, first_head, stream):
    import numpy as np
    import torch

    dtype = NSP_F32 if src.dtype == torch.float32 else NSP_BF16
    if dst.dtype != src.dtype:
        raise ValueError("source and destination must have the same dtype")
    fh = np.ascontiguousarray(first_head, dtype=np.int32)
    rc = getattr(lib(), fn_name)(_ptr(src), _ptr(dst), int(tokens), int(heads), int(heads_per_block), len(fh),
                                 int(head_dim), dtype, fh.ctypes.data_as(ctypes.c_void_p), _stream_ptr(stream))
    if rc != NSP_OK:
        raise NspError(rc, fn_name)


def nsp_a2a_gather_heads(src, dst, tokens, heads, heads_per_block, head_dim, first_head, stream=None):
    """[tokens, heads, D] -> [len(first_head)][tokens, heads_per_block, D] (device tensors, flat or shaped)."""
    _a2a("nsp_a2a_gather_heads", src, dst, tokens, heads, heads_per_block, head_dim, first_head, stream)


def nsp_a2a_gather_heads_to(src, dst_tensors, dst_row, sample_off, tokens, heads, heads_per_block, head_dim, first_head,
                            stream=None):
    """The head gather fused with the exchange: block p is stored into dst_tensors[p] (the receiving GPU's packed
    attention buffer, or a local stand-in) at the rows dst_row[p, j] (device int64 [n_blocks, n_samples]) for the
    samples whose rows in src are given by sample_off (device int64 [n_samples + 1])."""
    import numpy as np
    import torch

    dtype = NSP_F32 if src.dtype == torch.float32 else NSP_BF16
    n = len(dst_tensors)
    fh = np.ascontiguousarray(first_head, dtype=np.int32)
    if len(fh) != n or any(t.dtype != src.dtype or not t.is_cuda for t in dst_tensors):
        raise ValueError("one destination tensor of the source's dtype per block")
    if dst_row.dtype != torch.int64 or sample_off.dtype != torch.int64 or not dst_row.is_cuda or not sample_off.is_cuda:
        raise ValueError("dst_row and sample_off are int64 device tensors")
    n_samples = sample_off.numel() - 1
    if dst_row.numel() != n * n_samples:
        raise ValueError("dst_row holds one row per (block, sample)")
    bases = (ctypes.c_void_p * n)(*[t.data_ptr() for t in dst_tensors])
    rc = lib().nsp_a2a_gather_heads_to(_ptr(src), bases, _ptr(dst_row.contiguous()), _ptr(sample_off.contiguous()),
                                       n_samples, int(tokens), int(heads), int(heads_per_block), n, int(head_dim), dtype,
                                       fh.ctypes.data_as(ctypes.c_void_p), _stream_ptr(stream))
    if rc != NSP_OK:
        raise NspError(rc, "nsp_a2a_gather_heads_to")


def nsp_a2a_scatter_heads(src, dst, tokens, heads, heads_per_block, head_dim, first_head, stream=None):
    """[len(first_head)][tokens, heads_per_block, D] -> [tokens, heads, D], adding blocks that share a head."""
    _a2a("nsp_a2a_scatter_heads", src, dst, tokens, heads, heads_per_block, head_dim, first_head, stream)


def nsp_plan_recompute_ws_bytes(plan: Plan) -> int:
    n = ctypes.c_size_t()
    rc = lib().nsp_plan_recompute_ws_bytes(plan.handle, ctypes.byref(n))
    if rc != NSP_OK:
        raise NspError(rc, "nsp_plan_recompute_ws_bytes")
    return int(n.value)


def nsp_attn_bwd_recompute(plan: Plan, recompute, q, k, v, o, d_o, lse, dq, dk, dv, softmax_scale, ws, dq_dtype=None,
                           dkv_dtype=None, stream=None):
    """nsp_attn_bwd with per-segment flags (uint8 [n_seg], host): o and lse of a flagged segment are never read."""
    import numpy as np
    import torch

    recompute = np.ascontiguousarray(recompute, dtype=np.uint8)
    if recompute.shape != (plan.n_seg,):
        raise ValueError("recompute must have one entry per segment")
    if dq_dtype is None:
        dq_dtype = NSP_F32 if dq.dtype == torch.float32 else NSP_BF16
    if dkv_dtype is None:
        dkv_dtype = NSP_F32 if dk.dtype == torch.float32 else NSP_BF16
    _check_tensors("nsp_attn_bwd_recompute", plan,
                   _bwd_specs(plan, q, k, v, o, d_o, lse, dq, dk, dv, dq_dtype, dkv_dtype))
    _check_ws("nsp_attn_bwd_recompute", ws)
    ws_bytes = 0 if ws is None else ws.numel() * ws.element_size()
    rc = lib().nsp_attn_bwd_recompute(plan.handle, recompute.ctypes.data_as(ctypes.c_void_p), _ptr(q), _ptr(k), _ptr(v),
                                      _ptr(o), _ptr(d_o), _ptr(lse), _ptr(dq), _ptr(dk), _ptr(dv), dq_dtype, dkv_dtype,
                                      float(softmax_scale), _ptr(ws), ws_bytes, _stream_ptr(stream))
    if rc != NSP_OK:
        raise NspError(rc, "nsp_attn_bwd_recompute")


def nsp_selftest_wait_timeout(plan: Plan, limit_clk: int = 1_000_000, stream=None):
    """Let one bounded device-side wait run out on purpose; the plan's status word then holds NSP_ERR_DEVICE_TIMEOUT."""
    rc = lib().nsp_selftest_wait_timeout(plan.handle, int(limit_clk), _stream_ptr(stream))
    if rc != NSP_OK:
        raise NspError(rc, "nsp_selftest_wait_timeout")


def nsp_plan_set_wait_limit(plan: Plan, sm_clocks: int):
    rc = lib().nsp_plan_set_wait_limit(plan.handle, int(sm_clocks))
    if rc != NSP_OK:
        raise NspError(rc, "nsp_plan_set_wait_limit")


def nsp_checked_withhold_load(plan: Plan, enable: bool):
    """Checked build only: the next forward launch leaves out one V tile load (failure-detection test)."""
    if not hasattr(lib(), "nsp_checked_withhold_load"):
        raise NspError(NSP_ERR_UNSUPPORTED, "nsp_checked_withhold_load (needs libnsp_checked.so)")
    rc = lib().nsp_checked_withhold_load(plan.handle, int(bool(enable)))
    if rc != NSP_OK:
        raise NspError(rc, "nsp_checked_withhold_load")


def nsp_device_status(plan: Plan):
    out = (ctypes.c_int32 * 4)()
    rc = lib().nsp_device_status(plan.handle, out)
    if rc != NSP_OK:
        raise NspError(rc, "nsp_device_status")
    return tuple(out)


def nsp_plan_set_profiling(plan: Plan, enable: bool):
    rc = lib().nsp_plan_set_profiling(plan.handle, int(bool(enable)))
    if rc != NSP_OK:
        raise NspError(rc, "nsp_plan_set_profiling")


def nsp_plan_kernel_ms(plan: Plan, kernel_id: int) -> float:
    ms = ctypes.c_float()
    rc = lib().nsp_plan_kernel_ms(plan.handle, kernel_id, ctypes.byref(ms))
    if rc != NSP_OK:
        raise NspError(rc, "nsp_plan_kernel_ms")
    return float(ms.value)


def nsp_attn_bwd_static(plan: Plan, q, k, v, o, d_o, lse, dq, dk, dv, softmax_scale, dq_dtype=None, dkv_dtype=None,
                        stream=None):
    """nsp_attn_bwd for callers that may not allocate: no workspace argument, the scratch is a fixed array inside
    the library (at most NSP_STATIC_WS_BYTES; larger batches raise NSP_ERR_WORKSPACE). Calls sharing a device
    must not overlap. Make the first call on a device outside any stream capture."""
    import torch

    if dq_dtype is None:
        dq_dtype = NSP_F32 if dq.dtype == torch.float32 else NSP_BF16
    if dkv_dtype is None:
        dkv_dtype = NSP_F32 if dk.dtype == torch.float32 else NSP_BF16
    _check_tensors("nsp_attn_bwd_static", plan,
                   _bwd_specs(plan, q, k, v, o, d_o, lse, dq, dk, dv, dq_dtype, dkv_dtype))
    rc = lib().nsp_attn_bwd_static(plan.handle, _ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(d_o), _ptr(lse), _ptr(dq),
                                   _ptr(dk), _ptr(dv), dq_dtype, dkv_dtype, float(softmax_scale), _stream_ptr(stream))
    if rc != NSP_OK:
        raise NspError(rc, "nsp_attn_bwd_static")
