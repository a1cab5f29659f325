"""Pins for the oracle's tile planner: brute-force enumeration + Python's sort, closed-form counts, the
identity sum(cost_fwd) == sum(cost_bwd) (both count visited (q tile, kv tile, q head) triples), and a
hand-enumerated fixture."""
import os

import numpy as np
import pytest

import oracle
from paper_2609_22755_b200 import workloads as W


def _brute(cu, hq, hkv, bm, bn):
    """Enumerate visited (q tile m, kv tile n) pairs directly from the causal mask, then derive items."""
    fwd, bwd = [], []
    for s in range(len(hq)):
        L = int(cu[s + 1] - cu[s])
        G = hq[s] // hkv[s]
        Mt, Nt = -(-L // bm), -(-L // bn)
        visits = np.zeros((Mt, Nt), bool)
        for m in range(Mt):
            for n in range(Nt):
                # tile (m, n) holds an unmasked pair iff its smallest key index <= its largest valid query index
                visits[m, n] = n * bn <= min(L, (m + 1) * bm) - 1
        for h in range(hq[s]):
            for m in range(Mt):
                fwd.append((s, h, m, int(visits[m].sum())))
        for g in range(hkv[s]):
            for n in range(Nt):
                bwd.append((s, g, n, int(G * visits[:, n].sum())))
    key = lambda it: (-it[3], it[0], it[2], it[1])
    return sorted(fwd, key=key), sorted(bwd, key=key)


CASES = [
    ([300, 0, 128], [2, 2, 4], [1, 1, 4]),
    ([1, 17, 127, 129, 255, 1000], [8, 8, 4, 4, 16, 16], [2, 2, 1, 1, 16, 16]),
    ([64, 128, 256, 512], [8] * 4, [2] * 4),
    ([5000, 77, 2049], [4, 32, 32], [1, 4, 4]),
]


@pytest.mark.parametrize("lengths,hq,hkv", CASES)
@pytest.mark.parametrize("bm,bn", [(128, 128), (256, 128), (128, 64), (64, 128)])
def test_matches_bruteforce_enumeration(lengths, hq, hkv, bm, bn):
    cu = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    bf, bb = _brute(cu, hq, hkv, bm, bn)
    f = oracle.plan_tiles(cu, hq, hkv, bm, bn, 0)
    b = oracle.plan_tiles(cu, hq, hkv, bm, bn, 1)
    assert [tuple(x) for x in f.tolist()] == bf
    assert [tuple(x) for x in b.tolist()] == bb
    # both lists count the same (q tile, kv tile, q head) visits
    assert f[:, 3].sum() == b[:, 3].sum()
    # keys are distinct -> the order is unique
    assert len({(x[0], x[1], x[2]) for x in f.tolist()}) == len(f)


@pytest.mark.parametrize("idx", [1, 2, 3, 4, 5, 6])
def test_counts_and_cost_sums_on_benchmark_configs(idx):
    w = W.config(idx)
    L = w.lengths
    Mt = -(-L // 128)
    f = oracle.plan_tiles(w.cu_seqlens, w.hq, w.hkv, 128, 128, 0)
    b = oracle.plan_tiles(w.cu_seqlens, w.hq, w.hkv, 128, 128, 1)
    assert len(f) == int((Mt * w.hq).sum())
    assert len(b) == int((Mt * w.hkv).sum())
    assert int(f[:, 3].astype(np.int64).sum()) == int((w.hq * Mt * (Mt + 1) // 2).sum())  # bm == bn closed form
    assert int(b[:, 3].astype(np.int64).sum()) == int(f[:, 3].astype(np.int64).sum())
    assert np.all(np.diff(f[:, 3]) <= 0) and np.all(np.diff(b[:, 3]) <= 0)


def test_hand_enumerated_fixture():
    path = os.path.join(os.path.dirname(__file__), "golden", "plan_tiny.txt")
    want = {}
    for line in open(path):
        line = line.split("#")[0].strip()
        if line:
            k, rest = line.split("=")
            want[k.strip()] = [tuple(int(x) for x in it.split()) for it in rest.split("|")]
    cu, hq, hkv = [0, 300, 300, 428], [2, 2, 4], [1, 1, 4]
    assert [tuple(x) for x in oracle.plan_tiles(cu, hq, hkv, 128, 128, 0).tolist()] == want["fwd"]
    assert [tuple(x) for x in oracle.plan_tiles(cu, hq, hkv, 128, 128, 1).tolist()] == want["bwd"]
    assert [tuple(x) for x in oracle.plan_tiles(cu, hq, hkv, 128, 128, 2).tolist()] == want["bwd_exec"]
    cu2, hq2, hkv2 = [0, 128, 428, 728], [2, 2, 4], [2, 1, 2]
    assert [tuple(x) for x in oracle.plan_tiles(cu2, hq2, hkv2, 128, 128, 1).tolist()] == want["bwd2"]
    assert [tuple(x) for x in oracle.plan_tiles(cu2, hq2, hkv2, 128, 128, 2).tolist()] == want["bwd2_exec"]


def _brute_exec(cu, hq, hkv, bm, bn):
    """The executed backward order written out as nested loops (no sort): lengths from the longest down, for equal
    lengths the segments in index order, kv heads, key tiles; the cost of an item counted from the causal mask."""
    L = [int(cu[s + 1] - cu[s]) for s in range(len(hq))]
    out = []
    for length in sorted(set(L), reverse=True):
        for s in range(len(hq)):
            if L[s] != length or length == 0:
                continue
            G = hq[s] // hkv[s]
            Mt, Nt = -(-length // bm), -(-length // bn)
            for g in range(hkv[s]):
                for n in range(Nt):
                    visits = sum(1 for m in range(Mt) if n * bn <= min(length, (m + 1) * bm) - 1)
                    out.append((s, g, n, G * visits))
    return out


@pytest.mark.parametrize("lengths,hq,hkv", CASES + [([300, 128, 300, 0, 300, 128], [4, 2, 2, 2, 8, 4], [2, 1, 2, 2, 2, 4])])
@pytest.mark.parametrize("bm,bn", [(128, 128), (256, 128), (128, 64)])
def test_executed_backward_order_matches_nested_loops(lengths, hq, hkv, bm, bn):
    cu = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    e = oracle.plan_tiles(cu, hq, hkv, bm, bn, 2)
    assert [tuple(x) for x in e.tolist()] == _brute_exec(cu, hq, hkv, bm, bn)
    # the same items as the published list
    b = oracle.plan_tiles(cu, hq, hkv, bm, bn, 1)
    assert sorted(map(tuple, e.tolist())) == sorted(map(tuple, b.tolist()))
