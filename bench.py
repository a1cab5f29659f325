#!/usr/bin/env python
"""Benchmark of the hot path: packed variable-length causal GQA attention, forward + backward, on the
nested-plan per-GPU shard (one 393,216-token segment at degree 8 next to a degree-1 long-tailed tail).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config 1..5]

One "step" = nsp_attn_fwd + nsp_attn_bwd over the whole batch. Prints ONE JSON line (rank 0).
  value     causal TFLOP/s fwd+bwd (14 * D * causal pairs * q heads per step), inputs resident in HBM
  e2e       the same metric with pinned-host -> device copies of Q,K,V,dO and device -> host copies of
            O,LSE,dQ,dK,dV inside the timed region, through the package's public API
  roofline  the dominant kernel (backward main) against the measured dense bf16 tensor peak
  cpu_baseline  the fp64 oracle timed on the host cores on a bounded sample (reported, not a target)
N > 1 (launched by torch.distributed.run): independent replicas, one shard per GPU with its own seed, no
data-path collective ("weak" scaling); time = max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time
from pathlib import Path

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

import numpy as np  # noqa: E402

from paper_2609_22755_b200 import workloads as W  # noqa: E402

METRIC = "causal attention TFLOP/s fwd+bwd on 1 B200 and % of dense BF16 roofline"
UNIT = "TFLOP/s"


def captured_traffic(kernel: str, workload: str):
    """dram__bytes_read.sum + dram__bytes_write.sum of one launch of `kernel` on `workload`, from the ncu capture
    summaries kept as text under profiles/ (lines `traffic <kernel> <workload> <bytes> ...`); None when no capture
    covers that pair."""
    f = ROOT / "profiles" / "dram_traffic.txt"
    if not f.exists():
        return None
    for line in f.read_text().splitlines():
        parts = line.split()
        if len(parts) >= 4 and parts[0] == "traffic" and parts[1] == kernel and parts[2] == workload:
            return int(float(parts[3]))
    return None


def measured_peaks():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        d = json.loads(p.read_text())
        return {"burst": float(d["bf16_tflops"]), "sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                "hbm_gbs": float(d["hbm_gbs"]), "source": "measured"}
    return {"burst": 1590.0, "sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


def cpu_sample(w: W.Workload) -> W.Workload:
    """Bounded sample of a workload for the CPU oracle: the first tokens of every segment (a prefix of a causal
    sequence is itself a valid causal problem), long segments cut to 6144 tokens, the others to 1536."""
    L = w.lengths
    longest = int(L.max()) if len(L) else 0
    cut = [min(int(x), 6144 if int(x) == longest else 1536) for x in L]
    return W.custom(cut, w.hq.tolist(), w.hkv.tolist(), seed=w.seed, name=w.name + "_cpu_sample")


def run_oracle_sample(w: W.Workload):
    import oracle

    ws = cpu_sample(w)
    t = W.make_tensors(ws)
    b = {n: W.bf16_bits(t[n]) for n in ("q", "k", "v", "do")}
    t0 = time.perf_counter()
    oracle.attn_fwd(b["q"], b["k"], b["v"], ws.cu_seqlens, ws.hq, ws.hkv, ws.head_dim, ws.softmax_scale)
    oracle.attn_bwd(b["q"], b["k"], b["v"], b["do"], ws.cu_seqlens, ws.hq, ws.hkv, ws.head_dim, ws.softmax_scale)
    dt = time.perf_counter() - t0
    flops = sum(ws.flops())
    desc = (f"first min(L,1536) tokens of every segment (6144 of the longest): {ws.n_seg} segments, "
            f"{int(ws.lengths.sum())} tokens, {flops / 1e12:.3f} TFLOP, fp64, {dt:.1f} s")
    return flops / dt / 1e12, dt, oracle.num_threads(), desc


def peaks_in_run(torch):
    """The two roofline denominators measured again in this process, the way the stored measured peaks were taken:
    a bf16 matmul of 8192^3 (best of 10 = burst) and a copy of 2^30 bf16 elements (read + write bytes, best of 10)."""
    dev = torch.device("cuda")
    ev = lambda: torch.cuda.Event(enable_timing=True)
    a = torch.randn(8192, 8192, device=dev, dtype=torch.bfloat16)
    b = torch.randn(8192, 8192, device=dev, dtype=torch.bfloat16)
    for _ in range(3):
        torch.matmul(a, b)
    best = float("inf")
    for _ in range(10):
        e0, e1 = ev(), ev()
        e0.record()
        torch.matmul(a, b)
        e1.record()
        e1.synchronize()
        best = min(best, e0.elapsed_time(e1))
    tflops = 2 * 8192 ** 3 / (best * 1e-3) / 1e12
    del a, b
    x = torch.empty(1 << 30, device=dev, dtype=torch.bfloat16)
    y = torch.empty_like(x)
    for _ in range(2):
        y.copy_(x)
    best = float("inf")
    for _ in range(10):
        e0, e1 = ev(), ev()
        e0.record()
        y.copy_(x)
        e1.record()
        e1.synchronize()
        best = min(best, e0.elapsed_time(e1))
    gbs = 2 * x.numel() * 2 / (best * 1e-3) / 1e9
    del x, y
    torch.cuda.empty_cache()
    return {"bf16_tflops": tflops, "hbm_gbs": gbs, "how": "torch.matmul bf16 8192^3 best of 10; copy of 2^30 bf16 best of 10"}


def short_segment_roofline(torch, B, peaks, lengths=(32, 128, 512), iters=5):
    """The HBM-bound class: uniform batches of 131,072 tokens at 32q/4kv in segments of L tokens; achieved algorithmic
    bytes per second of the forward launch and of the backward launches against the measured copy bandwidth."""
    out = {}
    dev = torch.device("cuda")
    for L in lengths:
        n = 131072 // L
        w = W.custom([L] * n, 32, 4, seed=7, name=f"uniform_{n}x{L}_32q4kv")
        qe, kve, le = w.q_elems(), w.kv_elems(), w.lse_elems()
        bf = torch.bfloat16
        q, do = (torch.randn(qe, device=dev, dtype=torch.float32).to(bf) for _ in range(2))
        k, v = (torch.randn(kve, device=dev, dtype=torch.float32).to(bf) for _ in range(2))
        o, dq = torch.empty_like(q), torch.empty_like(q)
        lse = torch.empty(le, device=dev, dtype=torch.float32)
        dk, dv = (torch.empty(kve, device=dev, dtype=torch.float32) for _ in range(2))
        plan = B.nsp_plan_tiles(w.cu_seqlens, w.hq, w.hkv, w.head_dim)
        ws = torch.empty(max(plan.bwd_ws_bytes, 256), dtype=torch.uint8, device=dev)
        fwd = lambda: B.nsp_attn_fwd(plan, q, k, v, o, lse, w.softmax_scale)
        bwd = lambda: B.nsp_attn_bwd(plan, q, k, v, o, do, lse, dq, dk, dv, w.softmax_scale, ws)

        def timed(fn):
            for _ in range(3):
                fn()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(iters):
                fn()
            e1.record()
            e1.synchronize()
            return e0.elapsed_time(e1) / iters

        t_f, t_b = timed(fwd), timed(bwd)
        bytes_f = 2 * (qe + 2 * kve) + 2 * qe + 4 * le                     # read Q,K,V; write O, LSE
        bytes_b = 2 * (3 * qe + 2 * kve) + 4 * le + 8 * le + 2 * qe + 8 * kve   # read Q,K,V,O,dO,LSE; delta w+r; dQ bf16, dK/dV fp32
        ff, fb = w.flops()
        out[f"L{L}"] = {
            "workload": w.name, "fwd_ms": t_f, "bwd_ms": t_b, "fwd_gbs": bytes_f / t_f / 1e6, "bwd_gbs": bytes_b / t_b / 1e6,
            "fwd_frac": bytes_f / t_f / 1e6 / peaks["hbm_gbs"], "bwd_frac": bytes_b / t_b / 1e6 / peaks["hbm_gbs"],
            "fwd_tflops": ff / t_f / 1e9, "bwd_tflops": fb / t_b / 1e9, "algorithmic_bytes": [bytes_f, bytes_b],
        }
        plan.destroy()
        del q, do, k, v, o, dq, lse, dk, dv, ws
        torch.cuda.empty_cache()
    return {"bound": "hbm", "peak": peaks["hbm_gbs"], "unit": "GB/s", "peak_kind": f"hbm_gbs of {peaks['source']}",
            "note": "bwd = all launches of the backward pass (first-tile kernel; preprocess, main and postprocess where a "
                    "segment has more than one tile); at L = 32 four segments share a tile", **out}


class ClockSampler:
    """nvidia-smi clocks line sampled every 200 ms while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_id: str):
        """gpu_id: what nvidia-smi -i takes; the device's UUID, because nvidia-smi numbers the GPUs of the machine,
        not the ones CUDA_VISIBLE_DEVICES leaves to this process."""
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(gpu_id), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "200"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
                pw.append(float(parts[2]))
            except ValueError:
                continue
            for nm, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "power_w_max": max(pw), "samples": len(sm),
                "reasons": sorted(reasons)}


def reference_arm(args, rank, world):
    """The oracle as it stands, timed on the host cores; each step is one bounded sample of the workload."""
    if rank != 0:
        return
    w = rank_workload(args.config, args.uniform, 0)
    vals = []
    for _ in range(args.warmup):
        run_oracle_sample(w)
    info = None
    for _ in range(args.steps):
        info = run_oracle_sample(w)
        vals.append(info)
    tf = statistics.mean(v[0] for v in vals)
    ms = statistics.mean(v[1] for v in vals) * 1e3
    line = {
        "impl": "reference", "metric": METRIC, "value": tf, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "note": "CPU oracle on a bounded sample of the workload"},
        "cpu_baseline": {"value": tf, "unit": UNIT, "cores": info[2], "kind": "oracle", "sample": info[3]},
        "e2e": {"value": tf, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def rank_workload(config: int, uniform: int, rank: int):
    """The shard a rank runs: every GPU gets the same configuration with its own seed (lengths and values), so N
    GPUs are N independent replicas and the job's work grows with N (weak scaling)."""
    if uniform > 0:
        n = max(1, 131072 // uniform)
        return W.custom([uniform] * n, 32, 4, seed=1000 * rank, name=f"uniform_{n}x{uniform}_32q4kv")
    if config == 0:
        return W.profile_case()
    if config == 7:
        return W.profile_case_large_head()
    return W.config(config, seed=(config - 1) + 1000 * rank)


def max_over_ranks(ms: float, world: int, device: str) -> float:
    """The step time of the job is the slowest rank's."""
    if world <= 1:
        return ms
    import torch
    import torch.distributed as dist

    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(flops_per_rank: float, world: int, ms: float) -> float:
    """TFLOP/s of the whole job: what all ranks processed divided by the slowest rank's time."""
    return world * flops_per_rank / (ms * 1e-3) / 1e12


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=4,
                    help="benchmark configuration 1..5 (default 4: the nested-plan shard); 6 = the mixed-degree "
                         "full-tree shard; 0 and 7 = the scaled-down nested and large-head cases used for profiler captures")
    ap.add_argument("--uniform", type=int, default=0, metavar="L",
                    help="instead of --config: 131,072 tokens at 32q/4kv in segments of L tokens each (short-segment "
                         "studies; not a bench value)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the in-run re-measurement of the peaks and the short-segment (HBM-bound) roofline lines")
    ap.add_argument("--profile-mode", action="store_true",
                    help="for runs under a profiler: allows fewer than 3 warm-up steps; the printed line is not a bench value")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        reference_arm(args, rank, world)
        return
    if not args.profile_mode:
        args.warmup = max(args.warmup, 3)

    # The CPU baseline is timed first, in a process of its own that never touches CUDA: it is the reference arm of
    # this script run for one untimed and one timed step, so the two arms report the same figure.
    cpu = None
    if world == 1 and rank == 0 and not args.no_cpu_baseline:
        # the untimed pass matters: on the GPU hosts the first pass of a fresh process takes twice as long as the later ones
        cmd = [sys.executable, str(Path(__file__).resolve()), "--impl", "reference", "--steps", "1", "--warmup", "1",
               "--config", str(args.config)] + (["--uniform", str(args.uniform)] if args.uniform else [])
        r = subprocess.run(cmd, capture_output=True, text=True)
        try:
            cpu = json.loads(r.stdout.strip().splitlines()[-1])["cpu_baseline"]
        except Exception:
            cpu = {"value": None, "unit": UNIT, "cores": None, "kind": "oracle", "sample": "failed: " + r.stderr[-200:]}

    import torch
    import torch.distributed as dist

    from paper_2609_22755_b200 import binding as B
    from paper_2609_22755_b200.api import NspAttention

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    B.lib()
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # one shard per GPU: same configuration, its own seed (lengths and values)
    w = rank_workload(args.config, args.uniform, rank)
    host = W.make_tensors(w)
    host = {k: v.pin_memory() for k, v in host.items()}
    eng = NspAttention(w, device=f"cuda:{local_rank}")
    eng.load(host)
    torch.cuda.synchronize()
    B.nsp_plan_set_profiling(eng.plan, True)
    f_fwd, f_bwd = w.flops()
    flops = f_fwd + f_bwd

    for _ in range(args.warmup):
        eng.step_device()
    barrier()
    assert eng.status()[0] == 0, f"device status {eng.status()}"

    try:
        gpu_id = "GPU-" + str(torch.cuda.get_device_properties(local_rank).uuid)
    except Exception:
        gpu_id = str(local_rank)
    sampler = ClockSampler(gpu_id)
    launches0 = B.launch_count()
    k_fwd, k_bwd, k_pre, k_post, k_first, k_ffirst = [], [], [], [], [], []
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    # Per-kernel device times come from CUDA events the library records around each of its kernels on the launching
    # stream. Reading them waits for the step, which is free when a step takes hundreds of milliseconds; short steps
    # (the other configurations) are interrupted as little as possible: there only the first and the last step of the
    # timed region are read.
    read_every = False
    for i in range(args.steps):
        eng.step_device()
        if i == 0 or i == args.steps - 1 or read_every:
            k_fwd.append(B.nsp_plan_kernel_ms(eng.plan, B.KERNEL_FWD))
            k_pre.append(B.nsp_plan_kernel_ms(eng.plan, B.KERNEL_BWD_PRE))
            k_bwd.append(B.nsp_plan_kernel_ms(eng.plan, B.KERNEL_BWD_MAIN))
            k_post.append(B.nsp_plan_kernel_ms(eng.plan, B.KERNEL_BWD_POST))
            k_first.append(B.nsp_plan_kernel_ms(eng.plan, B.KERNEL_BWD_FIRST))
            k_ffirst.append(B.nsp_plan_kernel_ms(eng.plan, B.KERNEL_FWD_FIRST))
            if i == 0:
                read_every = k_fwd[0] + k_bwd[0] > 50.0
    e1.record()
    barrier()
    launches = B.launch_count() - launches0
    clocks = sampler.stop()
    ms = max_over_ranks(e0.elapsed_time(e1) / args.steps, world, "cuda")
    value = whole_job_value(flops, world, ms)
    assert eng.status()[0] == 0, f"device status {eng.status()}"

    # ---- end to end: host buffers in, host buffers out
    e2e = None
    if not args.no_e2e:
        host_out = eng.alloc_host_outputs()
        h2d, d2h = eng.step_host(host, host_out)
        barrier()
        e0.record()
        for _ in range(args.steps):
            h2d, d2h = eng.step_host(host, host_out)
        e1.record()
        barrier()
        ms_e2e = max_over_ranks(e0.elapsed_time(e1) / args.steps, world, "cuda")
        e2e = {"value": whole_job_value(flops, world, ms_e2e), "unit": UNIT, "h2d_bytes_per_step": int(h2d),
               "d2h_bytes_per_step": int(d2h), "ms_per_step": ms_e2e}

    if rank == 0:
        peaks = measured_peaks()
        extras = {}
        if world == 1 and not args.no_extras:
            del eng, host  # give the device memory back before the extra measurements
            torch.cuda.empty_cache()
            extras["peaks_in_run"] = peaks_in_run(torch)
            extras["roofline_short"] = short_segment_roofline(torch, B, peaks)
        bwd_ms = statistics.mean(k_bwd)
        achieved = f_bwd / (bwd_ms * 1e-3) / 1e12
        roofline = {
            "kernel": "bwd_kernel (backward main)", "bound": "tensor", "achieved": achieved, "peak": peaks["sustained"],
            "unit": "TFLOP/s", "frac": achieved / peaks["sustained"], "traffic": captured_traffic("bwd_kernel", w.name),
            "peak_kind": f"bf16_tflops_sustained of {peaks['source']} (kernel runs hundreds of ms inside a step)",
            "frac_of_burst_peak": achieved / peaks["burst"], "burst_peak": peaks["burst"],
            "launch_ms": bwd_ms, "flops_per_launch": f_bwd,
        }
        if clocks.get("sm_mhz") and clocks.get("sm_max_mhz"):
            # the same launch scaled to the maximum SM clock (time x median MHz / max MHz): what the kernel would reach
            # if the 1,000 W cap did not pull the clock down; a reading aid, not a measured number
            roofline["achieved_at_max_clock"] = achieved * clocks["sm_max_mhz"] / clocks["sm_mhz"]
        fwd_ms = statistics.mean(k_fwd)
        roofline_fwd = {
            "kernel": "fwd_kernel", "bound": "tensor", "achieved": f_fwd / (fwd_ms * 1e-3) / 1e12, "peak": peaks["sustained"],
            "unit": "TFLOP/s", "frac": f_fwd / (fwd_ms * 1e-3) / 1e12 / peaks["sustained"],
            "frac_of_burst_peak": f_fwd / (fwd_ms * 1e-3) / 1e12 / peaks["burst"], "launch_ms": fwd_ms,
            "flops_per_launch": f_fwd,
        }
        line = {
            **({"profile_mode": True} if args.profile_mode else {}),
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic",
            "config": {"workload": w.name, "segments": int(w.n_seg), "tokens": int(w.lengths.sum()),
                       "longest_segment": int(w.lengths.max()), "head_dim": w.head_dim, "note": w.note,
                       "grad_dtypes": "dQ bf16, dK/dV fp32", "l2": "inputs exceed L2 (no flush needed)",
                       "parallelism": "replicas" if world > 1 else "1 GPU"},
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline, "roofline_fwd": roofline_fwd, "cpu_baseline": cpu,
            "fraction_of_burst_peak": value / world / peaks["burst"],
            "fraction_of_sustained_peak": value / world / peaks["sustained"],
            "peaks": {"bf16_tflops_burst": peaks["burst"], "bf16_tflops_sustained": peaks["sustained"],
                      "hbm_gbs": peaks["hbm_gbs"], "source": peaks["source"]},
            **extras,
            "kernels_ms": {"fwd_first_tile": statistics.mean(k_ffirst), "fwd": statistics.mean(k_fwd),
                           "bwd_preprocess": statistics.mean(k_pre),
                           "bwd_first_tile": statistics.mean(k_first), "bwd_main": bwd_ms,
                           "bwd_postprocess": statistics.mean(k_post)},
            "tflops": {"fwd": f_fwd / ((statistics.mean(k_fwd) + statistics.mean(k_ffirst)) * 1e-3) / 1e12,
                       "bwd": f_bwd / ((statistics.mean(k_pre) + statistics.mean(k_first) + bwd_ms
                                        + statistics.mean(k_post)) * 1e-3) / 1e12},
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
