"""TEST INFRASTRUCTURE: ctypes front-end of the fp64 CPU oracle (``nsp_oracle.c``).

Only tests, the smoke check and the benchmark's CPU-baseline / reference legs import this package. It never
imports the CUDA package and shares nothing with it. The attention and tile-plan arithmetic lives in the C file;
this module compiles it with gcc, marshals numpy arrays and reshapes results. The one function written here in
plain Python loops are ``recompute_mark`` (the save / recompute walk of the paper's tree-level recomputation) and
``route_sp_tree`` (the paper's Algorithm 1, prefix-completion SP-tree routing) with its ``cost_table``.

Conventions (identical to the C file header): packed ragged token-major tensors, bf16 inputs passed as
``uint16`` bit patterns (or ``float64`` arrays for finite-difference checks), float64 outputs.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "nsp_oracle.c"
_LIB = _HERE / "liboracle.so"
_lib = None


def build(force: bool = False) -> Path:
    """Compile the oracle with gcc (-O2, OpenMP). Rebuilds when the source is newer than the library."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".tmp{os.getpid()}.so")
        cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-fno-fast-math", str(_SRC), "-o", str(tmp), "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(str(_LIB))
        _lib.orc_num_threads.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(_load().orc_num_threads())


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _i32(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _dt(a) -> int:
    if a.dtype == np.uint16:
        return 0
    if a.dtype == np.float64:
        return 1
    raise TypeError("oracle inputs are uint16 (bf16 bits) or float64")


def _check(rc: int, what: str):
    if rc != 0:
        raise RuntimeError(f"oracle {what} failed with code {rc}")


def layout_sizes(cu, hq, hkv, D):
    cu, hq, hkv = _i32(cu), _i32(hq), _i32(hkv)
    L = np.diff(cu).astype(np.int64)
    return int((L * hq).sum() * D), int((L * hkv).sum() * D), int((L * hq).sum())


def attn_fwd(q, k, v, cu, hq, hkv, D, scale):
    """Full forward. Returns (O [q_elems] f64, LSE [lse_elems] f64)."""
    lib = _load()
    cu, hq, hkv = _i32(cu), _i32(hq), _i32(hkv)
    qe, _, le = layout_sizes(cu, hq, hkv, D)
    O = np.zeros(qe, np.float64)
    LSE = np.zeros(le, np.float64)
    dt = _dt(q)
    rc = lib.orc_attn_fwd(_p(q), _p(k), _p(v), ctypes.c_int(dt), _p(cu), _p(hq), _p(hkv), ctypes.c_int(len(hq)),
                          ctypes.c_int(D), ctypes.c_double(scale), _p(O), _p(LSE))
    _check(rc, "attn_fwd")
    return O, LSE


def attn_bwd(q, k, v, d_o, cu, hq, hkv, D, scale, rows=None, want_dq=True):
    """Full backward (or, with rows=[(seg,row),...], the sums restricted to those query rows).

    Returns (dQ, dK, dV) as flat float64 arrays in the packed layout (dQ is None when want_dq is False).
    """
    lib = _load()
    cu, hq, hkv = _i32(cu), _i32(hq), _i32(hkv)
    qe, kve, _ = layout_sizes(cu, hq, hkv, D)
    dQ = np.zeros(qe, np.float64) if want_dq else None
    dK = np.zeros(kve, np.float64)
    dV = np.zeros(kve, np.float64)
    if rows is None:
        rs = ri = None
        n = 0
    else:
        rows = np.asarray(rows, dtype=np.int32).reshape(-1, 2)
        rs, ri = _i32(rows[:, 0]), _i32(rows[:, 1])
        n = len(rs)
    rc = lib.orc_attn_bwd(_p(q), _p(k), _p(v), _p(d_o), ctypes.c_int(_dt(q)), _p(cu), _p(hq), _p(hkv),
                          ctypes.c_int(len(hq)), ctypes.c_int(D), ctypes.c_double(scale), _p(rs), _p(ri),
                          ctypes.c_int64(n), _p(dQ), _p(dK), _p(dV))
    _check(rc, "attn_bwd")
    return dQ, dK, dV


def attn_rows(q, k, v, d_o, cu, hq, hkv, D, scale, samples):
    """O, LSE, dQ for sampled (seg, q head, row) triples. d_o may be None (then dQ is None)."""
    lib = _load()
    cu, hq, hkv = _i32(cu), _i32(hq), _i32(hkv)
    samples = np.asarray(samples, dtype=np.int32).reshape(-1, 3)
    n = len(samples)
    ss, sh, sr = _i32(samples[:, 0]), _i32(samples[:, 1]), _i32(samples[:, 2])
    O = np.zeros((n, D), np.float64)
    LSE = np.zeros(n, np.float64)
    dQ = np.zeros((n, D), np.float64) if d_o is not None else None
    rc = lib.orc_attn_rows(_p(q), _p(k), _p(v), _p(d_o), ctypes.c_int(_dt(q)), _p(cu), _p(hq), _p(hkv),
                           ctypes.c_int(len(hq)), ctypes.c_int(D), ctypes.c_double(scale), ctypes.c_int64(n), _p(ss),
                           _p(sh), _p(sr), _p(O), _p(LSE), _p(dQ))
    _check(rc, "attn_rows")
    return O, LSE, dQ


def attn_cols(q, k, v, d_o, cu, hq, hkv, D, scale, samples):
    """dK, dV for sampled (seg, kv head, column) triples under the full dO."""
    lib = _load()
    cu, hq, hkv = _i32(cu), _i32(hq), _i32(hkv)
    samples = np.asarray(samples, dtype=np.int32).reshape(-1, 3)
    n = len(samples)
    ss, sh, sc = _i32(samples[:, 0]), _i32(samples[:, 1]), _i32(samples[:, 2])
    dK = np.zeros((n, D), np.float64)
    dV = np.zeros((n, D), np.float64)
    rc = lib.orc_attn_cols(_p(q), _p(k), _p(v), _p(d_o), ctypes.c_int(_dt(q)), _p(cu), _p(hq), _p(hkv),
                           ctypes.c_int(len(hq)), ctypes.c_int(D), ctypes.c_double(scale), ctypes.c_int64(n), _p(ss),
                           _p(sh), _p(sc), _p(dK), _p(dV))
    _check(rc, "attn_cols")
    return dK, dV


def plan_tiles(cu, hq, hkv, bm=128, bn=128, pass_=0):
    """Sorted tile work list as an int32 array [n_items, 4] = (seg, head, tile, cost)."""
    lib = _load()
    cu, hq, hkv = _i32(cu), _i32(hq), _i32(hkv)
    n = ctypes.c_int64(0)
    rc = lib.orc_plan_tiles(_p(cu), _p(hq), _p(hkv), ctypes.c_int(len(hq)), ctypes.c_int(bm), ctypes.c_int(bn),
                            ctypes.c_int(pass_), None, ctypes.c_int64(0), ctypes.byref(n))
    _check(rc, "plan_tiles(size)")
    out = np.zeros((max(n.value, 1), 4), np.int32)
    rc = lib.orc_plan_tiles(_p(cu), _p(hq), _p(hkv), ctypes.c_int(len(hq)), ctypes.c_int(bm), ctypes.c_int(bn),
                            ctypes.c_int(pass_), _p(out), ctypes.c_int64(n.value), ctypes.byref(n))
    _check(rc, "plan_tiles")
    return out[: n.value]


def recompute_mark(lengths, hq, level, budget_bytes, head_dim=128):
    """Save / recompute marking of one GPU's segments (paper Sec. 4.2.2 "Tree-Level Recomputation"). The segments are
    visited level by level starting at the root; the bytes of attention output that saving a segment keeps alive are
    added up; the first segment that would exceed the budget ends the walk, and it and everything after it is
    recomputed. Inside a level the order is by recomputation cost, most expensive first.

    lengths, hq, level: one entry per segment (level: larger = closer to the root). A saved segment keeps its O
    slice (2 bytes per element) and its LSE (4 bytes per row) alive; its recomputation cost is hq * L(L+1)/2.
    Returns (flags, saved_bytes): flags[s] = 1 for recompute, 0 for save. Ties keep the segment order."""
    n = len(lengths)
    visit = []
    for lv in sorted(set(int(x) for x in level), reverse=True):  # root first
        members = [s for s in range(n) if int(level[s]) == lv]
        # inside a level: larger recomputation cost first; Python's sort is stable, so ties keep their order
        members.sort(key=lambda s: -(int(hq[s]) * (int(lengths[s]) * (int(lengths[s]) + 1) // 2)))
        visit += members
    flags = [1] * n
    used = 0
    for s in visit:
        need = int(lengths[s]) * int(hq[s]) * (2 * head_dim + 4)
        if used + need > budget_bytes:
            break  # the budget is reached: this segment and all later ones are recomputed
        used += need
        flags[s] = 0
    return np.asarray(flags, dtype=np.uint8), used


def route_sp_tree(lengths, cost, n_levels, k, w, b_tok, monotone=False):
    """Prefix-completion SP-tree routing (paper Algorithm 1), step by step in the paper's order.

    The SP tree is the full binary tree over P = 2**(n_levels-1) GPUs: node (l, i) covers GPUs
    [i * 2**l, (i + 1) * 2**l) and runs its samples at SP degree 2**l. cost[j][l] is the load the cost model
    attributes to EVERY GPU of a level-l node when sample j is placed there (any integer unit); the model is
    additive, so CostModel(a) is the per-GPU sum. Token loads follow the paper's Tok_p: a sample of length L on a
    degree-d node adds L / d to each of its GPUs; they are kept in units of 1/P token so that they stay integers.

    State S = (a, C, T). FeasibleNodes = all tree nodes, root first, left to right (with ``monotone``: no level
    above the level given to the previous, longer sample of the state). Beam and final choice break ties by order
    of generation. The tail goes to the leaves ("effective leaf units" = the single-GPU nodes).

    Returns None if the prefix search runs out of token-feasible states, else
    (level[j], index[j], C[p], T[p] in 1/P tokens, feasible) with feasible = every GPU within b_tok."""
    M = len(lengths)
    K = n_levels - 1
    P = 1 << K
    order = sorted(range(M), key=lambda j: -int(lengths[j]))  # stable: equal lengths keep their order
    H, R = order[:k], order[k:]
    Q = [({}, [0] * P, [0] * P, K)]  # (a, C, T, level of the last placed sample)
    for j in H:
        N = []
        for (a, C, T, last) in Q:
            for l in range(K, -1, -1):
                if monotone and l > last:
                    continue
                for i in range(P >> l):
                    a2 = dict(a)
                    a2[j] = (l, i)
                    C2, T2 = list(C), list(T)
                    for p in range(i << l, (i + 1) << l):
                        C2[p] += int(cost[j][l])
                        T2[p] += int(lengths[j]) * (P >> l)
                    if max(T2) <= b_tok * P:
                        N.append((a2, C2, T2, l))
        if not N:
            return None
        N.sort(key=lambda S: max(S[1]))  # stable
        Q = N[:w]
    done = []
    for (a, C, T, _) in Q:
        a, C, T = dict(a), list(C), list(T)
        for j in R:
            Lj = int(lengths[j])
            fits = [p for p in range(P) if T[p] + Lj * P <= b_tok * P]
            if fits:
                u = min(fits, key=lambda p: C[p])  # least-loaded unit that satisfies the budget (first on ties)
            else:
                u = min(range(P), key=lambda p: T[p])  # none does: the unit with the smallest token load
            a[j] = (0, u)
            C[u] += int(cost[j][0])
            T[u] += Lj * P
        done.append((a, C, T))
    feas = [S for S in done if max(S[2]) <= b_tok * P] if done else []
    pool = feas if feas else done
    a, C, T = min(pool, key=lambda S: max(S[1]))
    level = [a[j][0] for j in range(M)]
    index = [a[j][1] for j in range(M)]
    return level, index, C, T, bool(feas)


def cost_table(lengths, n_levels, hq, hkv, head_dim, tcomp_ns, link_gbs, other_ns_per_token):
    """The paper's hierarchical cost model (Sec. 4.1.2) for one sample on a level-l node, per covered GPU, forward +
    backward, in nanoseconds: SP-backend level = compute (causal pairs x local q heads x profiled ns per pair and
    head for the sample's length class) + prologue / epilogue all-to-alls (the (d-1)/d share of the GPU's L/d
    tokens; Q, K, V in and O out, both passes, bf16) over the level's link bandwidth; model level = non-attention
    time per resident token. tcomp_ns[l][b], b = clip(floor(log2 L), 5, 20) - 5. Returns int64 [n, n_levels]."""
    import math

    out = np.zeros((len(lengths), n_levels), dtype=np.int64)
    for j, L in enumerate(int(x) for x in lengths):
        b = min(max(L.bit_length() - 1, 5), 20) - 5 if L > 0 else 0
        pairs = L * (L + 1) / 2.0
        for l in range(n_levels):
            d = float(1 << l)
            comp = pairs * (hq / d) * float(tcomp_ns[l][b])
            comm = 0.0
            if l > 0:
                comm = (L / d) * ((d - 1.0) / d) * (4.0 * head_dim * (2.0 * hq + 2.0 * hkv)) / float(link_gbs[l])
            other = (L / d) * float(other_ns_per_token)
            out[j, l] = math.floor(comp + comm + other + 0.5)
    return out
