"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle on the same seeded inputs.

Small cases and scaled-down twins compare every element; the full-size benchmark configurations compare
sampled query rows (O, LSE, dQ), the last key columns (dK, dV under the full dO) and a sparse-dO probe (all of
dK, dV), each computed independently by the oracle. The tile work lists are compared bit for bit.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch

    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    import oracle
    import parity_util as P
    from paper_2609_22755_b200 import binding as B
    from paper_2609_22755_b200 import workloads as W

    B.lib()  # fails loudly if the extension is missing
    return dict(torch=torch, oracle=oracle, P=P, B=B, W=W)


def _full_case(env, w, **kw):
    P = env["P"]
    run = P.GpuRun(w, **kw)
    run.forward()
    run.backward()
    assert run.status()[0] == 0
    res = run.results()
    ref = P.oracle_full(w, run.host)
    return P.compare_full(w, res, ref), run, res, ref


@pytest.mark.parametrize("idx", [1, 2, 3, 4, 5, 6])
def test_tile_plan_bit_exact_full_size(env, idx):
    B, W, oracle = env["B"], env["W"], env["oracle"]
    w = W.config(idx)
    plan = B.nsp_plan_tiles(w.cu_seqlens, w.hq, w.hkv, w.head_dim)
    # pass 2 is the order the backward kernel walks (group-major); the oracle defines it independently
    for p in (0, 1, 2):
        got = B.nsp_plan_get(plan, p)
        want = oracle.plan_tiles(w.cu_seqlens, w.hq, w.hkv, 128, 128, p)
        assert got.dtype == np.int32 and got.shape == want.shape
        assert np.array_equal(got, want)
    plan.destroy()


def test_cfg1_every_element(env):
    _full_case(env, env["W"].config(1))


def test_ragged_tails_every_element(env):
    # lengths 1, 17, 127, 129, 255, 1000, 3 ..., a zero-length segment, MQA / GQA / MHA runs
    _full_case(env, env["W"].ragged())


@pytest.mark.parametrize("head_dim", [128, 64])
def test_short_segments_that_share_a_first_tile(env, head_dim):
    """Consecutive segments of fewer than 128 tokens inside a run go through the first-tile kernels as one tile
    (block-diagonal causal mask, per-segment LSE layout). Covered: packs of exactly 128 tokens (tile stores) and ragged
    ones, a pack of eight segments, a zero-length segment inside a pack, a 128-token and a multi-tile segment between
    packs, odd and unit group sizes; every element of every output against the oracle, and the published lists (which
    know nothing of packs) unchanged."""
    W, B, oracle = env["W"], env["B"], env["oracle"]
    lengths = [5, 60, 63, 1, 127, 2, 64, 64] + [100, 28, 128, 30, 98] + [200, 7, 0, 9, 112] + [16] * 8 + [48, 48, 48]
    hq = [8] * 8 + [3] * 5 + [4] * 5 + [16] * 11
    hkv = [2] * 8 + [1] * 5 + [4] * 5 + [2] * 11
    w = W.custom(lengths, hq, hkv, seed=21, name=f"shared_first_tiles_d{head_dim}", head_dim=head_dim)
    errs, run, res, ref = _full_case(env, w)
    for p_ in (0, 1, 2):
        assert np.array_equal(B.nsp_plan_get(run.plan, p_), oracle.plan_tiles(w.cu_seqlens, w.hq, w.hkv, 128, 128, p_))
    # uniform batches of very short segments: every tile holds 128 / L whole segments
    for L, n in ((16, 24), (48, 9)):
        _full_case(env, W.custom([L] * n, [8] * n, [2] * n, seed=22 + L, name=f"uniform_{L}_d{head_dim}", head_dim=head_dim))


def test_bf16_gradients_and_fp32_dq_variants(env):
    # the dtype arguments of nsp_attn_bwd: fp32 dQ meets the tolerance; bf16 dK/dV are produced and close
    # (their output rounding alone can exceed 2e-2 where |dV| > 8, so only rel-L2 is asserted for them)
    W, P = env["W"], env["P"]
    w = W.custom([300, 77], [8, 8], [2, 2], seed=5)
    _full_case(env, w, dq_dtype="f32", dkv_dtype="f32")
    run = P.GpuRun(w, dq_dtype="bf16", dkv_dtype="bf16")
    run.forward()
    run.backward()
    res, ref = run.results(), P.oracle_full(w, run.host)
    for n in ("dk", "dv"):
        assert P.errors(res[n], ref[n])[1] <= P.REL_L2_TOL


@pytest.mark.parametrize("idx", [2, 3, 4, 5, 6])
def test_scaled_down_twins_every_element(env, idx):
    _full_case(env, env["W"].config(idx, twin=True))


@pytest.mark.parametrize("case", ["cfg1", "ragged", 2, 3, 4, 5, 6])
def test_head_dim_64_every_element(env, case):
    """The same segment structures with head_dim = 64 (softmax scale 1/8): cfg1, the ragged case and the scaled-down
    twins, every element of every output against the oracle; the tile plan does not depend on the head dimension."""
    W, P, B, oracle = env["W"], env["P"], env["B"], env["oracle"]
    base = W.config(1) if case == "cfg1" else W.ragged() if case == "ragged" else W.config(case, twin=True)
    w = W.custom(base.lengths.tolist(), base.hq.tolist(), base.hkv.tolist(), seed=base.seed, name=base.name + "_d64",
                 head_dim=64)
    errs, run, res, ref = _full_case(env, w)
    for p_ in (0, 1, 2):
        assert np.array_equal(B.nsp_plan_get(run.plan, p_), oracle.plan_tiles(w.cu_seqlens, w.hq, w.hkv, 128, 128, p_))
    if case in ("ragged", 6):  # and through the recomputing backward, every second segment dropped
        torch = env["torch"]
        flags = (np.arange(w.n_seg) % 2).astype(np.uint8)
        qo, lo = w.q_offsets(), w.lse_offsets()
        for s_ in np.nonzero(flags)[0]:
            run.o[qo[s_]:qo[s_ + 1]] = float("nan")
            run.lse[lo[s_]:lo[s_ + 1]] = float("nan")
        ws = torch.empty(B.nsp_plan_recompute_ws_bytes(run.plan), dtype=torch.uint8, device=run.dev)
        B.nsp_attn_bwd_recompute(run.plan, flags, run.q, run.k, run.v, run.o, run.do, run.lse, run.dq, run.dk, run.dv,
                                 w.softmax_scale, ws)
        assert run.status()[0] == 0
        got = run.results()
        for name in ("dq", "dk", "dv"):
            P.check(f"{w.name}:recompute:{name}", got[name], ref[name])


def test_peaked_scores_exercise_the_rescale_path(env):
    """Q and K three times larger than in the benchmark data: scores spread over +-40 in log2 units, so the running
    maximum of a row keeps jumping by far more than the lazy-rescale threshold (2^8) from one key tile to the next.
    This exercises what N(0,1) data hardly ever reaches: the in-place rescale of O, and tiles exponentiated against
    a reference maximum that is one tile old (values of P far above 1). O and LSE keep the absolute tolerances.
    The gradients are larger here and, with nearly one-hot P on every row, carry the error of delta = dO.O taken
    from the bf16 O (the first-tile remedy of the kernel covers rows 0..127 only): they keep the relative-L2 bound,
    and their max-abs bound is 1 % of max|ref|."""
    W, P, torch = env["W"], env["P"], env["torch"]
    w = W.custom([1536, 700, 300, 129], [4, 4, 8, 2], [1, 1, 2, 2], seed=9, name="peaked")
    host = W.make_tensors(w)
    host["q"] = (host["q"].float() * 3.0).to(torch.bfloat16)
    host["k"] = (host["k"].float() * 3.0).to(torch.bfloat16)
    run = P.GpuRun(w, tensors=host)
    run.forward()
    run.backward()
    assert run.status()[0] == 0
    res = run.results()
    ref = P.oracle_full(w, run.host)
    P.check("peaked:o", res["o"], ref["o"])
    assert np.max(np.abs(res["lse"] - ref["lse"])) <= P.LSE_ABS_TOL * max(1.0, float(np.abs(ref["lse"]).max()) / 16)
    for n in ("dq", "dk", "dv"):
        ma, rl = P.check(f"peaked:{n}", res[n], ref[n], max_abs_tol=max(P.MAX_ABS_TOL, 1e-2 * float(np.abs(ref[n]).max())))
        print(f"peaked:{n} max-abs {ma:.4g} (max|ref| {np.abs(ref[n]).max():.3g}) rel-L2 {rl:.3g}")


@pytest.mark.parametrize("which", ["all", "budget", "alternate", "none"])
@pytest.mark.parametrize("case", ["full_tree_twin", "ragged"])
def test_backward_with_recomputation(env, case, which):
    """Tree-level recomputation: for the flagged segments O and LSE are poisoned with NaN before the backward call,
    which must recompute what it needs; the gradients are compared with the oracle element by element, and with the
    plain backward of the same run."""
    torch, P, B, W = env["torch"], env["P"], env["B"], env["W"]
    w = W.config(6, twin=True) if case == "full_tree_twin" else W.ragged()
    run = P.GpuRun(w)
    run.forward()
    run.backward()
    plain = {n: getattr(run, n).clone() for n in ("dq", "dk", "dv")}
    n = w.n_seg
    if which == "all":
        flags = np.ones(n, np.uint8)
    elif which == "none":
        flags = np.zeros(n, np.uint8)
    elif which == "alternate":
        flags = (np.arange(n) % 2).astype(np.uint8)
    else:  # the marking of an activation budget that holds about half of the shard's attention output
        total = int((w.lengths * w.hq).sum()) * (2 * w.head_dim + 4)
        level = (w.hq.max() // w.hq).astype(np.int32)  # SP degree of the segment's node
        flags, saved = B.nsp_recompute_mark(w.cu_seqlens, w.hq, level, total // 2)
        assert 0 < saved <= total // 2 and 0 < flags.sum() < n
    qo, lo = w.q_offsets(), w.lse_offsets()
    o, lse = run.o.clone(), run.lse.clone()
    for s in range(n):
        if flags[s]:
            o[qo[s]:qo[s + 1]] = float("nan")
            lse[lo[s]:lo[s + 1]] = float("nan")
    for t in (run.dq, run.dk, run.dv):
        t.fill_(float("nan"))
    ws = torch.empty(B.nsp_plan_recompute_ws_bytes(run.plan), dtype=torch.uint8, device=run.dev)
    B.nsp_attn_bwd_recompute(run.plan, flags, run.q, run.k, run.v, o, run.do, lse, run.dq, run.dk, run.dv,
                             w.softmax_scale, ws)
    assert run.status()[0] == 0
    res = run.results()
    ref = P.oracle_full(w, run.host)
    for name in ("dq", "dk", "dv"):
        P.check(f"{w.name}:recompute[{which}]:{name}", res[name], ref[name])
    if which == "none":  # nothing recomputed: the very same kernels on the very same inputs
        for name in ("dk", "dv"):
            assert torch.equal(getattr(run, name), plain[name])
    # too small a workspace is refused
    with pytest.raises(B.NspError):
        B.nsp_attn_bwd_recompute(run.plan, flags, run.q, run.k, run.v, o, run.do, lse, run.dq, run.dk, run.dv,
                                 w.softmax_scale, run.ws[:max(run.plan.bwd_ws_bytes - 256, 0)])
    if which == "alternate":  # the same through the user-facing wrapper
        from paper_2609_22755_b200.api import NspAttention

        eng = NspAttention(w)
        eng.load(run.host)
        eng.forward()
        eng.o.copy_(o)
        eng.lse.copy_(lse)
        eng.backward(recompute=flags)
        torch.cuda.synchronize()
        assert eng.status()[0] == 0
        for name in ("dk", "dv"):
            assert torch.equal(getattr(eng, name), getattr(run, name))


def test_host_to_host_step_equals_the_device_step(env):
    """The end-to-end call (nsp_attn_step_host through the C ABI: pinned host tensors in and out, device copies in a
    workspace of its own, the copies on the plan's second stream under the kernels) returns what
    the device-resident step leaves in the device buffers: O, LSE, dK, dV bit for bit, dQ (bf16, from the fp32
    accumulator) within one rounding of the fp32 sum. Two steps in a row, to cover the reuse of the buffers."""
    torch, W = env["torch"], env["W"]
    from paper_2609_22755_b200.api import NspAttention

    w = W.custom([1536, 700, 300, 129, 64], [4, 4, 8, 2, 2], [1, 1, 2, 2, 1], seed=13, name="host_step")
    host = {k: v.pin_memory() for k, v in W.make_tensors(w).items()}
    eng = NspAttention(w)
    eng.load(host)
    eng.step_device()
    torch.cuda.synchronize()
    want = {n: getattr(eng, n).cpu() for n in ("o", "lse", "dq", "dk", "dv")}
    for n in ("q", "k", "v", "do", "o", "lse", "dq", "dk", "dv"):
        getattr(eng, n).zero_()
    out = eng.alloc_host_outputs()
    for _ in range(2):
        for t in out.values():
            t.zero_()
        h2d, d2h = eng.step_host(host, out)
        torch.cuda.synchronize()
        assert eng.status()[0] == 0
        assert h2d == sum(host[n].numel() * host[n].element_size() for n in ("q", "k", "v", "do"))
        assert d2h == sum(t.numel() * t.element_size() for t in out.values())
        for n in ("o", "lse", "dk", "dv"):
            assert torch.equal(out[n], want[n]), n
        assert torch.allclose(out["dq"].float(), want["dq"].float(), rtol=2 ** -7, atol=1e-6)


def test_routed_shards_run_through_the_kernels(env):
    """Planner output instead of a hand-made shard: a scaled-down long-tailed batch is routed over eight GPUs (cost
    table from the shipped measured coefficients, Algorithm 1), and the shards of the first GPU and of the GPU with
    the most segments go through the kernels and are compared with the oracle element by element."""
    W = env["W"]
    from paper_2609_22755_b200 import planner

    tail = W.lognormal_lengths(3, 8 * 2048 - 12288, 48, 1.3, 16, 1024)
    lengths = [12288] + tail
    r = planner.route_batch(lengths, 4, 2300, prefix_k=6, beam_w=4)
    assert r["feasible"] and int(r["level"][0]) == 3
    shards = r["shards"]
    pick = {0, int(np.argmax([s.n_seg for s in shards]))}
    for p in sorted(pick):
        w = shards[p]
        assert w.n_seg >= 2 and int(w.hq[0]) == 4
        _full_case(env, w)


def test_one_gpu_of_a_routed_batch_with_recomputation(env):
    """The pieces in the order an iteration uses them, for the first GPU of an eight-GPU tree at reduced scale: route
    the batch (cost table, Algorithm 1), take the GPU's shard, mark its segments under an activation budget that
    holds the root segment only, run forward, drop O and LSE of the marked segments, run the recomputing backward,
    compare with the oracle."""
    torch, P, B, W = env["torch"], env["P"], env["B"], env["W"]
    from paper_2609_22755_b200 import planner

    tail = W.lognormal_lengths(7, 8 * 2048 - 12288, 48, 1.3, 16, 1024)
    lengths = [12288] + tail
    r = planner.route_batch(lengths, 4, 2300, prefix_k=6, beam_w=4)
    w = r["shards"][0]
    level = np.asarray([int(r["level"][j]) for j in r["sample_ids"][0]], dtype=np.int32)
    root_bytes = int(w.lengths[0]) * int(w.hq[0]) * (2 * w.head_dim + 4)
    flags, saved = B.nsp_recompute_mark(w.cu_seqlens, w.hq, level, root_bytes)
    assert saved == root_bytes and flags[0] == 0 and flags[1:].all()
    run = P.GpuRun(w)
    run.forward()
    qo, lo = w.q_offsets(), w.lse_offsets()
    for s in np.nonzero(flags)[0]:
        run.o[qo[s]:qo[s + 1]] = float("nan")
        run.lse[lo[s]:lo[s + 1]] = float("nan")
    ws = torch.empty(B.nsp_plan_recompute_ws_bytes(run.plan), dtype=torch.uint8, device=run.dev)
    B.nsp_attn_bwd_recompute(run.plan, flags, run.q, run.k, run.v, run.o, run.do, run.lse, run.dq, run.dk, run.dv,
                             w.softmax_scale, ws)
    assert run.status()[0] == 0
    res, ref = run.results(), P.oracle_full(w, run.host)
    for name in ("dq", "dk", "dv"):
        P.check(f"{w.name}:{name}", res[name], ref[name])


def test_bounded_wait_runs_out_and_is_reported(env):
    """Failure detection without a fault: a one-warp kernel waits on a barrier nothing arrives at; the library's
    bounded wait gives up, the status word carries the record, the plan refuses further work, and the context is
    still good for another plan."""
    B, W, P = env["B"], env["W"], env["P"]
    w = W.config(1)
    run = P.GpuRun(w)
    B.nsp_selftest_wait_timeout(run.plan, 1_000_000)
    # the failing kernel writes its record to mapped host memory: once it has run, the very next call on the plan
    # refuses, without anybody having polled nsp_device_status
    env["torch"].cuda.synchronize()
    with pytest.raises(B.NspError) as e:
        run.forward()
    assert e.value.code == B.NSP_ERR_DEVICE_TIMEOUT
    with pytest.raises(B.NspError) as e:
        run.backward()
    assert e.value.code == B.NSP_ERR_DEVICE_TIMEOUT
    code, item, where, aux = B.nsp_device_status(run.plan)
    assert (code, item, where, aux) == (B.NSP_ERR_DEVICE_TIMEOUT, -1, 90, 1_000_000 >> 10)
    _full_case(env, w)  # a fresh plan on the same context runs and matches the oracle


def test_empty_and_degenerate_batches(env):
    B, W, P, torch = env["B"], env["W"], env["P"], env["torch"]
    # no segments at all
    plan = B.nsp_plan_tiles([0], [], [], 128)
    assert plan.q_elems == 0 and len(B.nsp_plan_get(plan, 0)) == 0 and len(B.nsp_plan_get(plan, 1)) == 0
    B.nsp_attn_fwd(plan, None, None, None, None, None, 0.1)
    B.nsp_attn_bwd(plan, None, None, None, None, None, None, None, None, None, 0.1, None, dq_dtype=0, dkv_dtype=1)
    plan.destroy()
    # only zero-length segments
    plan = B.nsp_plan_tiles([0, 0, 0], [4, 8], [2, 2], 128)
    assert plan.q_elems == 0 and len(B.nsp_plan_get(plan, 0)) == 0
    plan.destroy()
    # 1-token segments: O = V exactly (bf16 copy), dQ = dK = 0 up to rounding, dV = sum of the group's dO
    w = W.custom([1, 1, 1], [4, 4, 2], [2, 2, 1], seed=3)
    run = P.GpuRun(w)
    run.forward()
    run.backward()
    res = run.results()
    v = run.host["v"].float().numpy().astype(np.float64)
    o = res["o"].reshape(-1, 128)
    exp_rows = []
    kvo = 0
    for s in range(w.n_seg):
        G = w.hq[s] // w.hkv[s]
        for h in range(w.hq[s]):
            exp_rows.append(v[kvo + (h // G) * 128: kvo + (h // G + 1) * 128])
        kvo += w.hkv[s] * 128
    assert np.array_equal(o, np.stack(exp_rows))
    # dS = P (dP - delta) vanishes up to the rounding of P = exp2(s - lse) ~ 1
    assert np.max(np.abs(res["dq"])) <= 1e-4 and np.max(np.abs(res["dk"])) <= 1e-4
    do = run.host["do"].float().numpy().astype(np.float64)
    qo, kvo = w.q_offsets(), w.kv_offsets()
    for s in range(w.n_seg):
        G = w.hq[s] // w.hkv[s]
        want = do[qo[s]:qo[s + 1]].reshape(w.hkv[s], G, 128).sum(axis=1)
        assert np.max(np.abs(res["dv"][kvo[s]:kvo[s + 1]].reshape(w.hkv[s], 128) - want)) <= 2e-2


def test_argument_errors_on_device(env):
    B, W, P, torch = env["B"], env["W"], env["P"], env["torch"]
    w = W.config(1)
    run = P.GpuRun(w)
    with pytest.raises(B.NspError) as e:
        B.nsp_attn_fwd(run.plan, run.q, run.k, run.v, run.o, run.lse, -1.0)
    assert e.value.code == B.NSP_ERR_INVALID_ARG
    with pytest.raises(B.NspError) as e:
        B.nsp_attn_fwd(run.plan, run.q[1:], run.k, run.v, run.o, run.lse, 0.1)  # 2-byte offset: misaligned
    assert e.value.code == B.NSP_ERR_INVALID_ARG
    with pytest.raises(B.NspError) as e:
        B.nsp_attn_bwd(run.plan, run.q, run.k, run.v, run.o, run.do, run.lse, run.dq, run.dk, run.dv, 0.1, run.ws[:256])
    assert e.value.code == B.NSP_ERR_WORKSPACE
    with pytest.raises(B.NspError) as e:
        B.nsp_attn_bwd(run.plan, run.q, run.k, run.v, run.o, run.do, run.lse, run.dq, run.dk, run.dv, 0.1, run.ws,
                       dq_dtype=7)
    assert e.value.code == B.NSP_ERR_INVALID_ARG
    assert run.status() == (0, 0, 0, 0)


def test_packing_order_invariance_and_reproducibility(env):
    W, P, torch = env["W"], env["P"], env["torch"]
    lengths, hq, hkv = [700, 130, 2048, 64], [8, 8, 4, 4], [2, 2, 1, 1]
    w = W.custom(lengths, hq, hkv, seed=21)
    run = P.GpuRun(w)
    run.forward()
    run.backward()
    a = run.results()
    # same inputs again: O, LSE, dK, dV bitwise equal (fixed accumulation order). dQ tiles are added to the fp32
    # accumulator with floating-point reductions in arrival order: equal up to the rounding of an fp32 sum, which
    # shows in the fp32 output (1e-5 of the largest element), not at the parity tolerance
    run32 = P.GpuRun(w, tensors=run.host, dq_dtype="f32")
    dq32 = []
    for _ in range(2):
        run32.forward()
        run32.backward()
        dq32.append(run32.results()["dq"])
    assert np.max(np.abs(dq32[0] - dq32[1])) <= 1e-5 * np.max(np.abs(dq32[0]))
    run.forward()
    run.backward()
    b = run.results()
    for n in ("o", "lse", "dk", "dv"):
        assert np.array_equal(a[n], b[n]), n
    # bf16 dQ of two runs: at most one rounding step apart where an fp32 sum sits on a rounding boundary
    assert np.max(np.abs(a["dq"] - b["dq"]) / np.maximum(np.abs(a["dq"]), 1e-3)) <= 2.0 ** -7
    # permute the two runs (segments 2,3 first): every segment's results are unchanged
    qo, kvo, lo = w.q_offsets(), w.kv_offsets(), w.lse_offsets()
    perm = [2, 3, 0, 1]
    wp = W.custom([lengths[p] for p in perm], [hq[p] for p in perm], [hkv[p] for p in perm], seed=21)
    host = {}
    for name, off in (("q", qo), ("do", qo), ("k", kvo), ("v", kvo)):
        host[name] = torch.cat([run.host[name][off[p]:off[p + 1]] for p in perm])
    runp = P.GpuRun(wp, tensors=host)
    runp.forward()
    runp.backward()
    c = runp.results()
    pqo, pkvo, plo = wp.q_offsets(), wp.kv_offsets(), wp.lse_offsets()
    for new, p in enumerate(perm):
        for n, off, poff in (("o", qo, pqo), ("lse", lo, plo), ("dk", kvo, pkvo), ("dv", kvo, pkvo)):
            assert np.array_equal(a[n][off[p]:off[p + 1]], c[n][poff[new]:poff[new + 1]]), (n, p)
        x, y = c["dq"][pqo[new]:pqo[new + 1]], a["dq"][qo[p]:qo[p + 1]]
        assert np.max(np.abs(x - y) / np.maximum(np.abs(y), 1e-3)) <= 2.0 ** -7


@pytest.mark.parametrize("mode", [True, "rounded"])
def test_deterministic_dq_option_is_bitwise_reproducible(env, mode):
    """Plan flags NSP_PLAN_DETERMINISTIC_DQ (the dQ tiles are added in key-tile order) and NSP_PLAN_ROUNDED_DQ (every
    term is rounded to a fixed quantum first, so that the fp32 sums are exact and their order is irrelevant): every
    output, dQ included, is bit for bit the same in three runs and under a permuted packing; and it still matches the
    oracle."""
    W, P, torch = env["W"], env["P"], env["torch"]
    lengths, hq, hkv = [3000, 130, 2048, 700, 64], [8, 8, 4, 4, 4], [2, 2, 1, 1, 1]
    w = W.custom(lengths, hq, hkv, seed=23)
    run = P.GpuRun(w, dq_dtype="f32", deterministic=mode)
    outs = []
    for _ in range(3):
        for t in (run.dq, run.dk, run.dv):
            t.fill_(float("nan"))
        run.forward()
        run.backward()
        assert run.status()[0] == 0
        outs.append(run.results())
    for n in ("o", "lse", "dq", "dk", "dv"):
        assert np.array_equal(outs[0][n], outs[1][n]) and np.array_equal(outs[0][n], outs[2][n]), n
    P.compare_full(w, outs[0], P.oracle_full(w, run.host))
    qo, kvo, lo = w.q_offsets(), w.kv_offsets(), w.lse_offsets()
    perm = [2, 3, 4, 0, 1]
    wp = W.custom([lengths[p] for p in perm], [hq[p] for p in perm], [hkv[p] for p in perm], seed=23)
    host = {}
    for name, off in (("q", qo), ("do", qo), ("k", kvo), ("v", kvo)):
        host[name] = torch.cat([run.host[name][off[p]:off[p + 1]] for p in perm])
    runp = P.GpuRun(wp, tensors=host, dq_dtype="f32", deterministic=mode)
    runp.forward()
    runp.backward()
    c = runp.results()
    pqo, pkvo, plo = wp.q_offsets(), wp.kv_offsets(), wp.lse_offsets()
    for new, p in enumerate(perm):
        for n, off, poff in (("o", qo, pqo), ("lse", lo, plo), ("dq", qo, pqo), ("dk", kvo, pkvo), ("dv", kvo, pkvo)):
            assert np.array_equal(outs[0][n][off[p]:off[p + 1]], c[n][poff[new]:poff[new + 1]]), (n, p)


def _sample_rows(w, rng, per_seg):
    rows = []
    for s in range(w.n_seg):
        L = int(w.lengths[s])
        if L == 0:
            continue
        cand = {0, L - 1, min(127, L - 1), min(128, L - 1), L // 2, max(0, L - 129), (L // 128) * 128 - 1 if L >= 128 else 0}
        cand |= set(int(x) for x in rng.integers(0, L, size=per_seg))
        for i in sorted(cand):
            rows.append((s, int(rng.integers(0, w.hq[s])), i))
    return rows


@pytest.mark.parametrize("idx,per_seg,last_cols", [(2, 2, 32), (3, 3, 32), (4, 6, 48), (5, 3, 24), (6, 3, 32)])
def test_full_size_configs_sampled(env, idx, per_seg, last_cols):
    """Full benchmark sizes in the launch configuration the benchmark times."""
    W, P, oracle, torch = env["W"], env["P"], env["oracle"], env["torch"]
    w = W.config(idx)
    run = P.GpuRun(w)
    run.forward()
    run.backward()
    assert run.status()[0] == 0
    torch.cuda.synchronize()
    bits = {n: W.bf16_bits(run.host[n]) for n in ("q", "k", "v", "do")}
    rng = np.random.default_rng(100 + idx)
    D = w.head_dim
    qo, kvo, lo = w.q_offsets(), w.kv_offsets(), w.lse_offsets()
    # only the long segments keep the oracle cost bounded: sample rows in the 4 longest + 4 random segments
    order = np.argsort(-w.lengths)
    keep = set(order[:4].tolist()) | set(rng.choice(w.n_seg, size=min(4, w.n_seg), replace=False).tolist())
    rows = [r for r in _sample_rows(w, rng, per_seg) if r[0] in keep]
    O, LSE, dQ = oracle.attn_rows(bits["q"], bits["k"], bits["v"], bits["do"], w.cu_seqlens, w.hq, w.hkv, D,
                                  w.softmax_scale, rows)
    idx_q = np.concatenate([qo[s] + (i * w.hq[s] + h) * D + np.arange(D) for s, h, i in rows])
    idx_l = np.array([lo[s] + h * w.lengths[s] + i for s, h, i in rows])
    go = run.o[torch.as_tensor(idx_q, device=run.dev)].float().cpu().numpy()
    gdq = run.dq[torch.as_tensor(idx_q, device=run.dev)].float().cpu().numpy()
    glse = run.lse[torch.as_tensor(idx_l, device=run.dev)].cpu().numpy()
    P.check(f"{w.name}:o[rows]", go, O.ravel())
    P.check(f"{w.name}:dq[rows]", gdq, dQ.ravel())
    assert np.max(np.abs(glse - LSE)) <= P.LSE_ABS_TOL
    # last key columns of the longest and of one short segment, every kv head of it
    cols = []
    for s in (int(order[0]), int(order[min(3, w.n_seg - 1)])):
        L = int(w.lengths[s])
        for g in range(min(int(w.hkv[s]), 2)):
            cols += [(s, g, j) for j in range(max(0, L - last_cols), L)]
    dK, dV = oracle.attn_cols(bits["q"], bits["k"], bits["v"], bits["do"], w.cu_seqlens, w.hq, w.hkv, D,
                              w.softmax_scale, cols)
    idx_kv = np.concatenate([kvo[s] + (j * w.hkv[s] + g) * D + np.arange(D) for s, g, j in cols])
    gdk = run.dk[torch.as_tensor(idx_kv, device=run.dev)].float().cpu().numpy()
    gdv = run.dv[torch.as_tensor(idx_kv, device=run.dev)].float().cpu().numpy()
    P.check(f"{w.name}:dk[last cols]", gdk, dK.ravel())
    P.check(f"{w.name}:dv[last cols]", gdv, dV.ravel())
    # gradient identities at full size (no oracle run needed): sum_j dK_j = 0, sum_j dV_j = sum of the group's dO
    s0 = int(order[0])
    L, Hkv, Hq = int(w.lengths[s0]), int(w.hkv[s0]), int(w.hq[s0])
    dk0 = run.dk[kvo[s0]:kvo[s0 + 1]].view(L, Hkv, D).double()
    dv0 = run.dv[kvo[s0]:kvo[s0 + 1]].view(L, Hkv, D).double()
    do0 = run.do[qo[s0]:qo[s0 + 1]].view(L, Hkv, Hq // Hkv, D).double()
    scale_ref = float(dk0.abs().sum(dim=0).max())
    assert float(dk0.sum(dim=0).abs().max()) <= 2e-3 * max(scale_ref, 1.0)
    want = do0.sum(dim=(0, 2))
    got = dv0.sum(dim=0)
    assert float((got - want).abs().max()) <= 2e-3 * float(dv0.abs().sum(dim=0).max())


@pytest.mark.parametrize("idx", [2, 3, 4, 5, 6])
def test_full_size_sparse_dO_probe(env, idx):
    """dO non-zero on a sparse set of query rows: every element of dK and dV then depends on those rows only,
    so the oracle can produce ALL of dK/dV of the full-size configuration; dQ must vanish off the rows."""
    W, P, oracle, torch = env["W"], env["P"], env["oracle"], env["torch"]
    w = W.config(idx)
    host = W.make_tensors(w)
    rng = np.random.default_rng(7 + idx)
    qo, kvo = w.q_offsets(), w.kv_offsets()
    D = w.head_dim
    order = np.argsort(-w.lengths)
    active = []
    for s, cnt in ((int(order[0]), 20), (int(order[1]), 8), (int(order[-1]), 4)):
        L = int(w.lengths[s])
        pick = {L - 1, 0, min(L - 1, 128)} | set(int(x) for x in rng.integers(0, L, size=cnt))
        active += [(s, i) for i in sorted(pick)]
    do = torch.zeros_like(host["do"])
    for s, i in active:
        a, b = qo[s] + i * w.hq[s] * D, qo[s] + (i + 1) * w.hq[s] * D
        do[a:b] = host["do"][a:b]
    host["do"] = do
    run = P.GpuRun(w, tensors=host)
    run.forward()
    run.backward()
    assert run.status()[0] == 0
    bits = {n: W.bf16_bits(host[n]) for n in ("q", "k", "v", "do")}
    _, dK, dV = oracle.attn_bwd(bits["q"], bits["k"], bits["v"], bits["do"], w.cu_seqlens, w.hq, w.hkv, D,
                                w.softmax_scale, rows=active, want_dq=False)
    P.check(f"{w.name}:dk[sparse dO, all]", run.dk.cpu().numpy(), dK)
    P.check(f"{w.name}:dv[sparse dO, all]", run.dv.cpu().numpy(), dV)
    del dK, dV
    gdq = run.dq.float()
    mask = torch.ones(w.q_elems(), dtype=torch.bool, device=run.dev)
    for s, i in active:
        mask[qo[s] + i * w.hq[s] * D: qo[s] + (i + 1) * w.hq[s] * D] = False
    assert float(gdq[mask].abs().max()) == 0.0
    rows = [(s, int(rng.integers(0, w.hq[s])), i) for s, i in active]
    _, _, dQ = oracle.attn_rows(bits["q"], bits["k"], bits["v"], bits["do"], w.cu_seqlens, w.hq, w.hkv, D,
                                w.softmax_scale, rows)
    idx_q = np.concatenate([qo[s] + (i * w.hq[s] + h) * D + np.arange(D) for s, h, i in rows])
    P.check(f"{w.name}:dq[active rows]", gdq[torch.as_tensor(idx_q, device=run.dev)].cpu().numpy(), dQ.ravel())


@pytest.mark.parametrize("L,hq", [(393216, 4), (131072, 16)])
def test_full_size_identical_keys_closed_form(env, L, hq):
    """The long segments of the nested shards (393,216 tokens at 4q/1kv, 131,072 at 16q/1kv) with IDENTICAL keys:
    then P_ij = 1/(i+1) and everything has a closed form that costs O(L*D) on the host (fp64, numpy):
    O_i = prefix mean of V, LSE_i = scale*q_i.k + ln(i+1), dQ = 0, dV_j = sum_h sum_{i>=j} dO_ih/(i+1),
    dK_j = scale*(A_j V_j - b_j) with suffix sums A_j = sum Q_ih dO_ih^T/(i+1), b_j = sum (dO_ih.O_i) Q_ih/(i+1).
    Every element of O, LSE, dQ, dV is compared, dK on sampled columns (first, last, tile edges, random). This is
    the case that exercises the longest accumulation chains of dK / dV (every key tile, ~100,000 tensor-core
    additions per accumulator element for the first keys)."""
    W, P, torch = env["W"], env["P"], env["torch"]
    D = 128
    w = W.custom([L], hq, 1, seed=77, name=f"identical_keys_{L}x{hq}")
    g = torch.Generator().manual_seed(77)
    rnd = lambda *shape: torch.randn(*shape, generator=g, dtype=torch.float32).to(torch.bfloat16)
    q, do, v = rnd(L, hq, D), rnd(L, hq, D), rnd(L, 1, D)
    kvec = rnd(D)
    k = kvec.expand(L, 1, D).contiguous()
    host = {"q": q.reshape(-1), "k": k.reshape(-1), "v": v.reshape(-1), "do": do.reshape(-1)}
    run = P.GpuRun(w, tensors=host)
    run.forward()
    run.backward()
    assert run.status()[0] == 0
    res = run.results()
    scale = w.softmax_scale
    inv = 1.0 / np.arange(1, L + 1, dtype=np.float64)                       # 1/(i+1)
    V = v.reshape(L, D).double().numpy()
    O = np.cumsum(V, axis=0) * inv[:, None]                                  # prefix mean, the same for every head
    P.check(f"{w.name}:o", res["o"].reshape(L, hq, D), np.broadcast_to(O[:, None, :], (L, hq, D)))
    kv = kvec.double().numpy()
    lse = scale * (q.reshape(L * hq, D).double().numpy() @ kv).reshape(L, hq) + np.log(np.arange(1, L + 1))[:, None]
    assert np.max(np.abs(res["lse"].reshape(hq, L) - lse.T)) <= P.LSE_ABS_TOL
    assert np.max(np.abs(res["dq"])) <= P.MAX_ABS_TOL                        # dQ = 0 exactly
    # dV_j = suffix sum over i of (sum_h dO_ih) / (i+1)
    dO = do.double().numpy()                                                 # [L, hq, D]
    Wd = dO.sum(axis=1) * inv[:, None]
    dV = np.cumsum(Wd[::-1], axis=0)[::-1]
    ma, rl = P.check(f"{w.name}:dv", res["dv"].reshape(L, D), dV)
    # b_j = suffix sum of sum_h (dO_ih . O_i) Q_ih / (i+1)
    Q = q.double().numpy()
    c = np.einsum("lhd,ld->lh", dO, O) * inv[:, None]                        # (dO_ih . O_i) / (i+1)
    b = np.cumsum(np.einsum("lh,lhd->ld", c, Q)[::-1], axis=0)[::-1]
    rng = np.random.default_rng(5)
    cols = sorted({0, 1, 5, 63, 127, 128, 129, 255, 256, 4095, 4096, L // 2, L - 129, L - 128, L - 2, L - 1}
                  | set(int(x) for x in rng.integers(0, L, size=16)))
    gdk = res["dk"].reshape(L, D)
    want = np.empty((len(cols), D))
    for t, j in enumerate(cols):
        # A_j V_j = sum_{i>=j} sum_h Q_ih (dO_ih . V_j) / (i+1)
        wgt = np.einsum("lhd,d->lh", dO[j:], V[j]) * inv[j:, None]
        want[t] = scale * (np.einsum("lh,lhd->d", wgt, Q[j:]) - b[j])
    mk, rk = P.check(f"{w.name}:dk[sampled cols]", gdk[cols], want)
    print(f"{w.name}: dV max-abs {ma:.4g} rel-L2 {rl:.3g}; dK max-abs {mk:.4g} rel-L2 {rk:.3g}")
