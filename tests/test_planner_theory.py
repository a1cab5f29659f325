"""Properties from the paper's appendices, checked on the planner (no device is touched).

Appendix A (pairing bound for SP doubling): with every sample forced onto the nodes of ONE tree level (= a static SP
degree s), the best critical load at degree 2s is never worse than at degree s, and the excess imbalance shrinks at least
by the factor (1 + rho) / 2, rho taken from the sorted group loads of the degree-s optimum. The planner is driven into
the static setting through its cost table (every other level priced out) and made exhaustive (full prefix, unbounded
beam), so the statement is tested on what the oracle and the library actually compute.

Appendix B (dyadic packing; laminar power-of-two groups relabel to SP-tree nodes): the constructive relabeling of the
proof is written out here and checked on random laminar families; the node -> GPU-range convention of the planner
(node (l, i) covers GPUs [i 2^l, (i + 1) 2^l)) is what it maps onto, and the plans the planner emits are laminar.
"""
import numpy as np
import pytest

import oracle


def _static_best(work, n_levels, level):
    """Best max-over-GPUs load when every sample must sit on a node of `level`, through the planner itself."""
    M = len(work)
    big = 10 ** 12
    # per-GPU load of sample j on a level-l node: its work divided evenly over the 2^l GPUs of the node
    cost = [[(w >> l) if l == level else big for l in range(n_levels)] for w in work]
    lengths = list(range(M, 0, -1))  # distinct, descending: the visiting order is the sample order
    out = oracle.route_sp_tree(lengths, cost, n_levels, M, 10 ** 9, 10 ** 9)
    assert out is not None
    lv, idx, C, T, feasible = out
    assert all(l == level for l in lv)
    return max(C), lv, idx, C


@pytest.mark.parametrize("seed", range(12))
def test_sp_doubling_never_worsens_the_best_imbalance_and_meets_the_pairing_bound(seed):
    rng = np.random.default_rng(seed)
    n_levels = 3  # P = 4 GPUs: degrees 1, 2, 4
    P = 1 << (n_levels - 1)
    M = int(rng.integers(3, 7))
    # long-tailed work, multiples of P so that the shares are integers
    work = [int(P * max(1, round(float(np.exp(rng.normal(3.0, 1.2)))))) for _ in range(M)]
    total = sum(work)
    for level in range(n_levels - 1):
        best_s, lv, idx, C = _static_best(work, n_levels, level)
        best_2s, _, _, _ = _static_best(work, n_levels, level + 1)
        mean = total / P  # per-GPU average, the same at every degree
        R_s, R_2s = best_s / mean, best_2s / mean
        assert R_2s <= R_s + 1e-12
        # group loads of the degree-s optimum (one entry per level-`level` node), sorted descending
        D = P >> level
        W = sorted((sum(w for j, w in enumerate(work) if idx[j] == q) for q in range(D)), reverse=True)
        Wbar = total / D
        if W[0] > Wbar:
            rho = (W[D // 2] - Wbar) / (W[0] - Wbar)
            assert -1.0 - 1e-12 <= rho <= 1.0 + 1e-12
            assert R_2s - 1.0 <= (1.0 + rho) / 2.0 * (R_s - 1.0) + 1e-9


def _dyadic_tile(sizes):
    """Appendix B, dyadic packing lemma, as an algorithm: power-of-two sizes summing to 2^k -> start offsets of aligned,
    pairwise disjoint intervals tiling [0, 2^k), in the order of `sizes`. Largest blocks first keeps every start aligned."""
    total = sum(sizes)
    assert total & (total - 1) == 0 and all(s & (s - 1) == 0 and s > 0 for s in sizes)
    order = sorted(range(len(sizes)), key=lambda t: -sizes[t])
    start, at = [0] * len(sizes), 0
    for t in order:
        assert at % sizes[t] == 0  # aligned: everything placed before is a multiple of this (smaller or equal) size
        start[t] = at
        at += sizes[t]
    return start


def _relabel(groups, K):
    """Appendix B, theorem: a laminar family of power-of-two-sized groups on 2^K workers -> a permutation pi of the
    workers under which every group becomes an aligned dyadic interval (the worker set of an SP-tree node)."""
    n = 1 << K
    fam = {frozenset(range(n))} | {frozenset([w]) for w in range(n)} | {frozenset(g) for g in groups}
    pi = {}

    def place(S, base):
        kids = [T for T in fam if T < S and not any(T < U < S for U in fam)]
        assert sum(len(T) for T in kids) == len(S)  # the singletons make the children cover S
        kids.sort(key=lambda T: (-len(T), min(T)))
        for T, off in zip(kids, _dyadic_tile([len(T) for T in kids])):
            if len(T) == 1:
                pi[next(iter(T))] = base + off
            else:
                place(T, base + off)

    place(frozenset(range(n)), 0)
    return pi


def _random_laminar(rng, K):
    """Random laminar family: pick tree nodes, then scramble the worker labels."""
    n = 1 << K
    nodes = [(l, i) for l in range(1, K) for i in range(n >> l) if rng.random() < 0.5]
    perm = rng.permutation(n)
    return [[int(perm[w]) for w in range(i << l, (i + 1) << l)] for l, i in nodes]


@pytest.mark.parametrize("seed", range(10))
def test_laminar_power_of_two_groups_relabel_to_tree_nodes(seed):
    rng = np.random.default_rng(100 + seed)
    K = int(rng.integers(2, 5))
    groups = _random_laminar(rng, K)
    pi = _relabel(groups, K)
    assert sorted(pi.values()) == list(range(1 << K))  # a bijection
    for g in groups:
        img = sorted(pi[w] for w in g)
        size = len(g)
        assert img == list(range(img[0], img[0] + size)) and img[0] % size == 0  # node (log2 size, img[0] / size)


def test_crossing_groups_are_not_laminar_and_cannot_be_relabelled():
    # {0,1} and {1,2}: power-of-two sizes, but they overlap without nesting; tree nodes are always nested or disjoint
    a, b = {0, 1}, {1, 2}
    assert a & b and not (a <= b or b <= a)
    with pytest.raises(AssertionError):
        _relabel([sorted(a), sorted(b)], 2)


@pytest.mark.parametrize("seed", range(6))
def test_planner_output_is_a_laminar_family_of_aligned_blocks(seed):
    rng = np.random.default_rng(200 + seed)
    n_levels = 4
    P = 1 << (n_levels - 1)
    M = int(rng.integers(4, 12))
    lengths = sorted((int(x) for x in rng.integers(8, 4000, M)), reverse=True)
    cost = [[(L * L) >> l for l in range(n_levels)] for L in lengths]
    out = oracle.route_sp_tree(lengths, cost, n_levels, min(M, 4), 3, 10 ** 9)
    assert out is not None
    lv, idx = out[0], out[1]
    ranges = [set(range(i << l, (i + 1) << l)) for l, i in zip(lv, idx)]
    assert all(max(r) < P for r in ranges)
    for x in ranges:
        for y in ranges:
            assert x <= y or y <= x or not (x & y)
