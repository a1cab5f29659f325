"""Routing (paper Sec. 4.1.2: cost model; Sec. 4.1.3: Algorithm 1): the oracle against exhaustive search, a textbook list
scheduler and invariants; the library's host functions against the oracle. No device is touched."""
import heapq
import itertools

import numpy as np
import pytest

import oracle


def _loads(lengths, cost, n_levels, level, index):
    """C_p and Tok_p (in 1/P tokens) of an assignment, from the definitions."""
    P = 1 << (n_levels - 1)
    C, T = [0] * P, [0] * P
    for j, (l, i) in enumerate(zip(level, index)):
        for p in range(P):
            if (p >> l) == i:
                C[p] += int(cost[j][l])
                T[p] += int(lengths[j]) * (P >> l)
    return C, T


def _nodes(n_levels):
    P = 1 << (n_levels - 1)
    return [(l, i) for l in range(n_levels) for i in range(P >> l)]


def _exhaustive(lengths, cost, n_levels, b_tok, monotone):
    """min over ALL assignments within the token budget of max_p C_p (None if there is none)."""
    P = 1 << (n_levels - 1)
    order = sorted(range(len(lengths)), key=lambda j: -lengths[j])
    best = None
    for combo in itertools.product(_nodes(n_levels), repeat=len(lengths)):
        lv = [c[0] for c in combo]
        if monotone and any(lv[order[t]] < lv[order[t + 1]] for t in range(len(order) - 1)):
            continue
        C, T = _loads(lengths, cost, n_levels, lv, [c[1] for c in combo])
        if max(T, default=0) <= b_tok * P:
            m = max(C, default=0)
            best = m if best is None else min(best, m)
    return best


def _instance(rng, M, n_levels):
    lengths = sorted((int(x) for x in rng.integers(1, 400, M)), reverse=True)
    rng.shuffle(lengths)
    # a plausible cost: quadratic compute shared by the group plus a per-level communication term
    cost = [[(L * L) // (1 << l) + (l * 37 * L) // (1 << l) + int(rng.integers(0, 5)) for l in range(n_levels)]
            for L in lengths]
    return lengths, cost


@pytest.mark.parametrize("seed", range(10))
@pytest.mark.parametrize("monotone", [False, True])
def test_full_prefix_and_unbounded_beam_is_exhaustive_search(seed, monotone):
    rng = np.random.default_rng(seed)
    n_levels = int(rng.integers(2, 4))  # P = 2 or 4
    M = int(rng.integers(1, 6 if n_levels == 2 else 5))
    lengths, cost = _instance(rng, M, n_levels)
    P = 1 << (n_levels - 1)
    for b_tok in (10**9, max(lengths), sum(lengths) // P + max(lengths) // 2, max(lengths) // 2):
        want = _exhaustive(lengths, cost, n_levels, b_tok, monotone)
        got = oracle.route_sp_tree(lengths, cost, n_levels, M, 10**9, b_tok, monotone)
        if want is None:
            assert got is None
            continue
        level, index, C, T, feasible = got
        assert feasible and max(C) == want
        assert (C, T) == _loads(lengths, cost, n_levels, level, index)


@pytest.mark.parametrize("seed", range(6))
def test_pure_tail_is_longest_first_list_scheduling(seed):
    """prefix 0, no budget: every sample goes to the least-loaded GPU, longest first (the textbook LPT rule)."""
    rng = np.random.default_rng(100 + seed)
    n_levels = 4
    lengths, cost = _instance(rng, 30, n_levels)
    level, index, C, T, feasible = oracle.route_sp_tree(lengths, cost, n_levels, 0, 3, 10**12)
    heap = [(0, p) for p in range(8)]
    want = {}
    for j in sorted(range(len(lengths)), key=lambda j: -lengths[j]):
        load, p = heapq.heappop(heap)
        want[j] = p
        heapq.heappush(heap, (load + cost[j][0], p))
    assert feasible and all(l == 0 for l in level)
    assert [want[j] for j in range(len(lengths))] == list(index)


def test_invariants_budget_fallback_and_infeasible_prefix():
    rng = np.random.default_rng(5)
    n_levels = 4
    P = 8
    lengths, cost = _instance(rng, 40, n_levels)
    for k, w, mono in [(0, 1, False), (4, 2, False), (8, 4, True), (12, 3, True)]:
        b_tok = sum(lengths) // P + max(lengths)
        level, index, C, T, feasible = oracle.route_sp_tree(lengths, cost, n_levels, k, w, b_tok, mono)
        assert (C, T) == _loads(lengths, cost, n_levels, level, index)
        assert sum(T) == P * sum(lengths)  # every sample's tokens are spread over its node exactly once
        assert feasible == (max(T) <= b_tok * P)
        order = sorted(range(len(lengths)), key=lambda j: -lengths[j])
        assert all(level[j] == 0 for j in order[k:])  # the tail sits on leaves
        if mono:
            lv = [level[j] for j in order[:k]]
            assert all(a >= b for a, b in zip(lv, lv[1:]))
    # a wider beam never loses to beam 1 on the searched prefix when there is no tail
    l8, c8 = lengths[:8], cost[:8]
    a = oracle.route_sp_tree(l8, c8, n_levels, 8, 1, 10**9)
    b = oracle.route_sp_tree(l8, c8, n_levels, 8, 64, 10**9)
    assert max(b[2]) <= max(a[2])
    # the longest sample cannot fit even on the root: the prefix search has no feasible state
    assert oracle.route_sp_tree([800, 10], [[1] * 4, [1] * 4], 4, 1, 2, 99) is None
    # a tail sample that fits nowhere goes to the leaf with the fewest tokens and the plan is flagged
    level, index, C, T, feasible = oracle.route_sp_tree([50, 40, 30], [[5, 5], [4, 4], [3, 3]], 2, 0, 1, 45)
    assert not feasible and list(index) == [0, 1, 1] and T == [100, 140]


def test_cost_table_closed_forms():
    tcomp = np.full((3, 16), 2e-3)
    link = np.array([0.0, 500.0, 250.0])
    c = oracle.cost_table([1000], 3, 32, 4, 128, tcomp, link, 7.0)[0]
    pairs = 1000 * 1001 // 2
    # level 0: no communication
    assert c[0] == round(pairs * 32 * 2e-3 + 1000 * 7.0)
    # degree 2: half the heads and tokens; half of the GPU's 500 tokens cross the link, 4*128*(64+8) bytes each
    assert c[1] == round(pairs * 16 * 2e-3 + 500 * 0.5 * 36864 / 500.0 + 500 * 7.0)
    assert c[2] == round(pairs * 8 * 2e-3 + 250 * 0.75 * 36864 / 250.0 + 250 * 7.0)
    # the length class selects the coefficient: only bucket floor(log2 4096) - 5 = 7 is non-zero here
    t2 = np.zeros((1, 16))
    t2[0, 7] = 1.0
    got = oracle.cost_table([4095, 4096, 8191, 8192, 31, 2**21], 1, 1, 1, 128, t2, [0.0], 0.0)[:, 0]
    assert list(got) == [0, 4096 * 4097 // 2, 8191 * 8192 // 2, 0, 0, 0]


@pytest.fixture(scope="module")
def B():
    from paper_2609_22755_b200 import build

    build.build_library()
    from paper_2609_22755_b200 import binding

    return binding


def test_library_routing_matches_the_oracle(B):
    rng = np.random.default_rng(11)
    n_inf = 0
    for trial in range(60):
        n_levels = int(rng.integers(1, 5))
        P = 1 << (n_levels - 1)
        M = int(rng.integers(0, 40))
        lengths, cost = _instance(rng, M, n_levels) if M else ([], np.zeros((0, n_levels), np.int64))
        k, w, mono = int(rng.integers(0, 7)), int(rng.integers(1, 9)), bool(rng.integers(0, 2))
        tight = (sum(lengths) // P + (max(lengths) if M else 0) // int(rng.integers(1, 4))) if M else 0
        b_tok = int(rng.choice([10**9, tight]))
        want = oracle.route_sp_tree(lengths, cost, n_levels, k, w, b_tok, mono)
        if want is None:
            n_inf += 1
            with pytest.raises(B.NspError) as e:
                B.nsp_route_sp_tree(lengths, np.asarray(cost).reshape(M, n_levels), n_levels, k, w, b_tok, mono)
            assert e.value.code == B.NSP_ERR_INFEASIBLE
            continue
        level, index, C, T, feasible = B.nsp_route_sp_tree(lengths, np.asarray(cost).reshape(M, n_levels), n_levels,
                                                           k, w, b_tok, mono)
        assert list(level) == list(want[0]) and list(index) == list(want[1])
        assert list(C) == want[2] and list(T) == want[3] and feasible == want[4]
    assert n_inf < 30


def test_library_cost_table_matches_the_oracle(B):
    rng = np.random.default_rng(2)
    lengths = [int(x) for x in rng.integers(0, 500000, 200)] + [0, 1, 31, 32, 63, 64, 2**20, 2**20 - 1]
    tcomp = rng.uniform(1e-4, 5e-3, (4, 16))
    link = np.array([0.0, 770.0, 770.0, 400.0])
    got = B.nsp_cost_table(lengths, 4, 32, 4, 128, tcomp, link, 11.5)
    want = oracle.cost_table(lengths, 4, 32, 4, 128, tcomp, link, 11.5)
    assert got.shape == want.shape and np.max(np.abs(got - want)) <= 1  # both round the same fp64 sum


def test_library_rejects_bad_arguments(B):
    with pytest.raises(B.NspError):
        B.nsp_route_sp_tree([5], np.array([[1, -1]]), 2, 1, 1, 10)
    with pytest.raises(B.NspError):
        B.nsp_route_sp_tree([5], np.array([[1, 1]]), 2, 1, 0, 10)
    with pytest.raises(B.NspError):
        B.nsp_cost_table([5], 2, 32, 4, 128, np.ones((2, 16)), np.array([0.0, 0.0]), 1.0)


def test_shards_from_routing():
    from paper_2609_22755_b200 import planner

    lengths = [4096, 1024, 512, 300, 0, 64]
    level = [2, 1, 1, 0, 0, 0]
    index = [0, 0, 1, 3, 1, 0]
    shards, ids = planner.shards_from_routing(lengths, level, index, 3, 32, 4)
    assert len(shards) == 4
    assert ids[0] == [0, 1, 5] and ids[1] == [0, 1] and ids[2] == [0, 2] and ids[3] == [0, 2, 3]
    w = shards[3]
    assert list(w.lengths) == [4096, 512, 300] and list(w.hq) == [8, 16, 32] and list(w.hkv) == [1, 2, 4]
    # every (sample, query head) pair is computed exactly once across the GPUs
    total = sum(int((s.lengths * s.hq).sum()) for s in shards)
    assert total == 32 * sum(lengths)


def test_route_batch_on_a_long_tailed_batch(B):
    """Eight GPUs, 65,536 tokens each: one 393,216-token sample plus a long tail, the shape of the nested-plan
    benchmark shard. The token budget forces the long sample onto the root; the measured cost table balances the
    rest."""
    from paper_2609_22755_b200 import planner
    from paper_2609_22755_b200 import workloads as W

    tail = W.lognormal_lengths(0, 8 * 65536 - 393216, 1024, 1.3, 16, 32768)
    lengths = [393216] + tail
    r = planner.route_batch(lengths, 4, 70000)
    assert r["feasible"] and int(r["level"][0]) == 3
    assert r["tok"].max() <= 70000 * 8 and int(r["tok"].sum()) == 8 * sum(lengths)
    load = r["load_ns"].astype(np.float64)
    assert load.max() / load.mean() < 1.01
    order = np.argsort(-np.asarray(lengths), kind="stable")
    lv = r["level"][order][:8]
    assert all(a >= b for a, b in zip(lv, lv[1:]))  # monotone SP over the searched prefix
    # greedy alone (no prefix search) cannot place the long sample and is far worse
    g = planner.route_batch(lengths, 4, 70000, prefix_k=0, beam_w=1)
    assert not g["feasible"] and g["load_ns"].max() > 5 * load.max()
    # GPU 0's shard: the long sample with 4 of the 32 query heads and one (replicated) KV head comes first
    w = r["shards"][0]
    assert int(w.lengths[0]) == 393216 and int(w.hq[0]) == 4 and int(w.hkv[0]) == 1
    assert sum(int((s.lengths * s.hq).sum()) for s in r["shards"]) == 32 * sum(lengths)
