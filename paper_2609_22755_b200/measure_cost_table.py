"""Measure the compute coefficients of the planner's cost model on the GPU at hand.

``python -m paper_2609_22755_b200.measure_cost_table --out cost_table.json`` times forward + backward of uniform
batches through the library for every SP level of a model (level l: hq / 2^l query heads and max(1, hkv / 2^l) KV
heads per GPU) and every length class b (segments of about 2^(b+5.5) tokens), and writes
``tcomp_ns[l][b]`` = nanoseconds per causal (query, key) pair and local query head, forward + backward: the profiled
compute throughput the paper's cost model takes as an input (Sec. 4.1.2, SP-backend level). Length classes whose batch
would exceed ``--max-pflop`` are not run; they take the value of the longest class that was (the time per pair no
longer changes there). Needs a CUDA device.
"""
from __future__ import annotations

import argparse
import json

import numpy as np

from . import binding as B
from . import workloads as W


def measure(hq=32, hkv=4, n_levels=4, tokens=131072, max_pflop=1.5, iters=3, device="cuda:0"):
    import torch

    dev = torch.device(device)
    table = np.zeros((n_levels, B.NSP_COST_BUCKETS))
    rows = []
    for l in range(n_levels):
        d = 1 << l
        hq_l, hkv_l = hq // d, max(1, hkv // d)
        last = None
        for b in range(B.NSP_COST_BUCKETS):
            L = int(round(2 ** (b + 5.5) / 16)) * 16
            n = max(1, tokens // L)
            w = W.custom([L] * n, hq_l, hkv_l, seed=b, name=f"level{l}_L{L}")
            f_fwd, f_bwd = w.flops()
            if (f_fwd + f_bwd) > max_pflop * 1e15 and last is not None:
                table[l, b] = last
                rows.append({"level": l, "bucket": b, "L": L, "segments": n, "extrapolated": True, "ns": last})
                continue
            g = torch.Generator(device=dev)
            g.manual_seed(b)
            rnd = lambda m: torch.randn(m, device=dev, generator=g, dtype=torch.float32).to(torch.bfloat16)
            q, do, k, v = rnd(w.q_elems()), rnd(w.q_elems()), rnd(w.kv_elems()), rnd(w.kv_elems())
            o = torch.empty_like(q)
            lse = torch.empty(w.lse_elems(), device=dev, dtype=torch.float32)
            dq = torch.empty_like(q)
            dk = torch.empty(w.kv_elems(), device=dev, dtype=torch.float32)
            dv = torch.empty_like(dk)
            plan = B.nsp_plan_tiles(w.cu_seqlens, w.hq, w.hkv, 128)
            ws = torch.empty(max(plan.bwd_ws_bytes, 256), dtype=torch.uint8, device=dev)

            def step():
                B.nsp_attn_fwd(plan, q, k, v, o, lse, w.softmax_scale)
                B.nsp_attn_bwd(plan, q, k, v, o, do, lse, dq, dk, dv, w.softmax_scale, ws)

            step()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(iters):
                step()
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / iters
            assert B.nsp_device_status(plan)[0] == 0
            ns = ms * 1e6 / (w.causal_pairs())  # causal_pairs already counts every local query head
            table[l, b] = last = ns
            rows.append({"level": l, "bucket": b, "L": L, "segments": n, "ms": ms, "ns": ns,
                         "tflops": (f_fwd + f_bwd) / ms / 1e9})
            plan.destroy()
            del q, do, k, v, o, lse, dq, dk, dv, ws
    return table, rows


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--out", required=True)
    ap.add_argument("--hq", type=int, default=32)
    ap.add_argument("--hkv", type=int, default=4)
    ap.add_argument("--levels", type=int, default=4)
    ap.add_argument("--max-pflop", type=float, default=1.5)
    args = ap.parse_args()
    import torch

    table, rows = measure(args.hq, args.hkv, args.levels, max_pflop=args.max_pflop)
    doc = {"what": "tcomp_ns[level][length class]: ns per causal (query, key) pair and local query head, forward + backward",
           "written_by": "python -m paper_2609_22755_b200.measure_cost_table",
           "device": torch.cuda.get_device_name(0), "model": {"hq": args.hq, "hkv": args.hkv, "head_dim": 128},
           "levels": args.levels, "buckets": B.NSP_COST_BUCKETS, "tcomp_ns": table.tolist(), "runs": rows}
    with open(args.out, "w") as f:
        json.dump(doc, f, indent=1)
    for r in rows:
        print(r)


if __name__ == "__main__":
    main()
