"""Save / recompute marking (paper Sec. 4.2.2 "Tree-Level Recomputation"): the oracle's walk against a hand-worked
fixture, against a brute-force definition on small random shards, and the library's host function against the
oracle. No device is touched."""
import itertools
import os

import numpy as np
import pytest

import oracle


def _fixture():
    path = os.path.join(os.path.dirname(__file__), "golden", "recompute_mark_tiny.txt")
    vals, cases = {}, []
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, rhs = [x.strip() for x in line.split("=", 1)]
        if key == "case":
            b, f, s = [x.strip() for x in rhs.split("|")]
            cases.append((int(b), [int(x) for x in f.split()], int(s)))
        else:
            vals[key] = [int(x) for x in rhs.split()]
    return vals, cases


def test_oracle_matches_the_hand_worked_fixture():
    vals, cases = _fixture()
    for budget, flags, saved in cases:
        got, used = oracle.recompute_mark(vals["lengths"], vals["hq"], vals["level"], budget)
        assert got.tolist() == flags, budget
        assert used == saved


def _brute(lengths, hq, level, budget, D=128):
    """The definition without the walk: among all prefixes of the visiting order (level descending, cost descending,
    index ascending), the longest one whose bytes fit; the order itself is found by trying all permutations."""
    n = len(lengths)
    cost = [hq[s] * (lengths[s] * (lengths[s] + 1) // 2) for s in range(n)]
    byt = [lengths[s] * hq[s] * (2 * D + 4) for s in range(n)]
    best = None
    for perm in itertools.permutations(range(n)):
        ok = all((level[a], cost[a], -a) >= (level[b], cost[b], -b) for a, b in zip(perm, perm[1:]))
        if ok:
            best = perm
            break
    k, used = 0, 0
    while k < n and used + byt[best[k]] <= budget:
        used += byt[best[k]]
        k += 1
    flags = [1] * n
    for s in best[:k]:
        flags[s] = 0
    return flags, used


@pytest.mark.parametrize("seed", range(12))
def test_oracle_matches_brute_force_on_small_shards(seed):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(1, 7))
    lengths = [int(x) for x in rng.choice([0, 16, 48, 128, 300, 1000], size=n)]
    hq = [int(x) for x in rng.choice([4, 8, 32], size=n)]
    level = [int(x) for x in rng.choice([1, 2, 4], size=n)]
    total = sum(l * h * 260 for l, h in zip(lengths, hq))
    for budget in [0, total // 3, total // 2, total - 1, total, total + 5] + [int(x) for x in rng.integers(0, total + 1, 4)]:
        budget = max(budget, 0)
        got, used = oracle.recompute_mark(lengths, hq, level, budget)
        want, wused = _brute(lengths, hq, level, budget)
        assert got.tolist() == want and used == wused


def test_oracle_invariants():
    rng = np.random.default_rng(7)
    n = 40
    lengths = rng.integers(0, 5000, n)
    hq = rng.choice([4, 8, 16, 32], n)
    level = rng.choice([1, 2, 4, 8], n)
    byt = lengths * hq * 260
    prev_saved = -1
    for budget in np.linspace(0, byt.sum() + 10, 23).astype(np.int64):
        flags, used = oracle.recompute_mark(lengths, hq, level, int(budget))
        assert used <= budget and used == int(byt[flags == 0].sum())
        assert used >= prev_saved  # a larger budget never saves less
        prev_saved = used
        # nothing is saved below something that is recomputed: every saved segment sits at a level >= every
        # recomputed one
        if (flags == 0).any() and (flags == 1).any():
            assert level[flags == 0].min() >= level[flags == 1].max()


@pytest.fixture(scope="module")
def B():
    from paper_2609_22755_b200 import build

    build.build_library()
    from paper_2609_22755_b200 import binding

    return binding


def test_library_matches_the_oracle(B):
    vals, cases = _fixture()
    cu = np.concatenate([[0], np.cumsum(vals["lengths"])])
    for budget, flags, saved in cases:
        got, used = B.nsp_recompute_mark(cu, vals["hq"], vals["level"], budget)
        assert got.tolist() == flags and used == saved
    rng = np.random.default_rng(3)
    for _ in range(20):
        n = int(rng.integers(0, 60))
        lengths = rng.integers(0, 9000, n)
        hq = rng.choice([4, 8, 16, 32, 64], n)
        level = rng.choice([1, 2, 4, 8, 16], n)
        cu = np.concatenate([[0], np.cumsum(lengths)])
        total = int((lengths * hq * 260).sum())
        for budget in [0, total // 2, total, int(rng.integers(0, total + 1))]:
            got, used = B.nsp_recompute_mark(cu, hq, level, budget)
            want, wused = oracle.recompute_mark(lengths, hq, level, budget)
            assert np.array_equal(got, want) and used == wused


def test_library_rejects_bad_arguments(B):
    with pytest.raises(B.NspError):
        B.nsp_recompute_mark([0, 10], [4], [1], -1)
    with pytest.raises(B.NspError):
        B.nsp_recompute_mark([0, 10, 5], [4, 4], [1, 1], 100)
    with pytest.raises(B.NspError):
        B.nsp_recompute_mark([0, 10], [0], [1], 100)
