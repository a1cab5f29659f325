"""Pins for the fp64 CPU oracle (forward, backward, sampled modes). No GPU, no CUDA library.

Each test checks the oracle against something other than itself: a second, structurally different evaluation
(dense L x L matrices with the explicit softmax Jacobian), central finite differences, closed forms, identities
of the definition, torch's CPU SDPA on the special case that reduces to it, and a hand-computed fixture.
"""
import os

import numpy as np
import pytest

import oracle

D_SMALL = 8


def _rand_problem(seed, lengths, hq, hkv, D):
    rng = np.random.default_rng(seed)
    lengths = np.asarray(lengths)
    cu = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    hq = np.asarray(hq, np.int32)
    hkv = np.asarray(hkv, np.int32)
    qe = int((lengths * hq).sum() * D)
    kve = int((lengths * hkv).sum() * D)
    q = rng.standard_normal(qe)
    k = rng.standard_normal(kve)
    v = rng.standard_normal(kve)
    do = rng.standard_normal(qe)
    return cu, hq, hkv, q, k, v, do


def _seg_views(cu, hq, hkv, D, q, k, v, do=None):
    """Yield per-segment dense views (Q [L,Hq,D], K, V [L,Hkv,D], dO) and flat offsets."""
    qo = kvo = lo = 0
    for s in range(len(hq)):
        L = int(cu[s + 1] - cu[s])
        nq, nkv = L * hq[s] * D, L * hkv[s] * D
        yield (s, L, q[qo:qo + nq].reshape(L, hq[s], D), k[kvo:kvo + nkv].reshape(L, hkv[s], D),
               v[kvo:kvo + nkv].reshape(L, hkv[s], D), None if do is None else do[qo:qo + nq].reshape(L, hq[s], D),
               qo, kvo, lo)
        qo += nq
        kvo += nkv
        lo += L * hq[s]


def _dense_reference(cu, hq, hkv, D, scale, q, k, v, do):
    """Second opinion: materialise P as an L x L matrix, form the softmax Jacobian diag(p) - p p^T of every row
    explicitly and apply the chain rule with matrix products."""
    O = np.zeros_like(q)
    dQ = np.zeros_like(q)
    dK = np.zeros_like(k)
    dV = np.zeros_like(k)
    LSE = np.zeros(int((np.diff(cu) * hq).sum()))
    for s, L, Q, K, V, dO, qo, kvo, lo in _seg_views(cu, hq, hkv, D, q, k, v, do):
        if L == 0:
            continue
        G = hq[s] // hkv[s]
        Os = np.zeros((L, hq[s], D))
        dQs = np.zeros((L, hq[s], D))
        dKs = np.zeros((L, hkv[s], D))
        dVs = np.zeros((L, hkv[s], D))
        mask = np.tril(np.ones((L, L), bool))
        for h in range(hq[s]):
            g = h // G
            S = scale * Q[:, h, :] @ K[:, g, :].T
            S = np.where(mask, S, -np.inf)
            E = np.exp(S - S.max(axis=1, keepdims=True))
            P = E / E.sum(axis=1, keepdims=True)
            LSE[lo + h * L: lo + (h + 1) * L] = np.log(E.sum(axis=1)) + S.max(axis=1)
            Os[:, h, :] = P @ V[:, g, :]
            dP = dO[:, h, :] @ V[:, g, :].T
            dS = np.zeros((L, L))
            for i in range(L):
                J = np.diag(P[i]) - np.outer(P[i], P[i])
                dS[i] = J @ dP[i]
            dQs[:, h, :] = scale * dS @ K[:, g, :]
            dKs[:, g, :] += scale * dS.T @ Q[:, h, :]
            dVs[:, g, :] += P.T @ dO[:, h, :]
        O[qo:qo + Os.size] = Os.ravel()
        dQ[qo:qo + Os.size] = dQs.ravel()
        dK[kvo:kvo + dKs.size] = dKs.ravel()
        dV[kvo:kvo + dKs.size] = dVs.ravel()
    return O, LSE, dQ, dK, dV


CASES = [
    ([5], [1], [1], 4),
    ([37], [4], [2], 8),
    ([1, 9, 0, 23], [4, 4, 4, 2], [1, 1, 1, 2], 8),
    ([16, 64], [8, 2], [2, 1], 16),
]


@pytest.mark.parametrize("lengths,hq,hkv,D", CASES)
def test_matches_dense_jacobian_reference(lengths, hq, hkv, D):
    cu, hq, hkv, q, k, v, do = _rand_problem(1, lengths, hq, hkv, D)
    scale = 0.37
    O, LSE = oracle.attn_fwd(q, k, v, cu, hq, hkv, D, scale)
    dQ, dK, dV = oracle.attn_bwd(q, k, v, do, cu, hq, hkv, D, scale)
    rO, rLSE, rdQ, rdK, rdV = _dense_reference(cu, hq, hkv, D, scale, q, k, v, do)
    for a, b in ((O, rO), (LSE, rLSE), (dQ, rdQ), (dK, rdK), (dV, rdV)):
        np.testing.assert_allclose(a, b, rtol=1e-11, atol=1e-12)


def test_gradients_match_central_finite_differences():
    D = D_SMALL
    cu, hq, hkv, q, k, v, do = _rand_problem(2, [11, 6], [4, 2], [2, 2], D)
    scale = 1.0 / np.sqrt(D)
    dQ, dK, dV = oracle.attn_bwd(q, k, v, do, cu, hq, hkv, D, scale)

    def loss(q_, k_, v_):
        O, _ = oracle.attn_fwd(q_, k_, v_, cu, hq, hkv, D, scale)
        return float((O * do).sum())

    h = 1e-5
    rng = np.random.default_rng(0)
    for arr, grad, which in ((q, dQ, 0), (k, dK, 1), (v, dV, 2)):
        idxs = rng.choice(arr.size, size=min(arr.size, 60), replace=False)
        for idx in idxs:
            args = [q.copy(), k.copy(), v.copy()]
            args[which][idx] += h
            up = loss(*args)
            args[which][idx] -= 2 * h
            dn = loss(*args)
            fd = (up - dn) / (2 * h)
            assert abs(fd - grad[idx]) <= 1e-7 * max(1.0, abs(grad[idx])), (which, idx, fd, grad[idx])


def test_one_token_segment_closed_form():
    # a 1-token sequence attends only to itself: O = V, LSE = scale*q.k, dV = sum of the group's dO, dQ = dK = 0
    D = 8
    cu, hq, hkv, q, k, v, do = _rand_problem(3, [1, 1], [4, 6], [2, 3], D)
    scale = 0.5
    O, LSE = oracle.attn_fwd(q, k, v, cu, hq, hkv, D, scale)
    dQ, dK, dV = oracle.attn_bwd(q, k, v, do, cu, hq, hkv, D, scale)
    for s, L, Q, K, V, dO, qo, kvo, lo in _seg_views(cu, hq, hkv, D, q, k, v, do):
        G = hq[s] // hkv[s]
        for h in range(hq[s]):
            g = h // G
            np.testing.assert_array_equal(O[qo + h * D: qo + (h + 1) * D], V[0, g])
            assert abs(LSE[lo + h] - scale * Q[0, h] @ K[0, g]) < 1e-14
        for g in range(hkv[s]):
            np.testing.assert_allclose(dV[kvo + g * D: kvo + (g + 1) * D], dO[0, g * G:(g + 1) * G].sum(axis=0),
                                       rtol=0, atol=1e-15)
    assert np.all(dQ == 0) and np.all(dK == 0)


def test_identical_keys_closed_form():
    # all keys equal: P_ij = 1/(i+1); O = causal prefix mean of V; LSE = scale*q.k + ln(i+1); dQ = 0;
    # dV_j = sum_h sum_{i>=j} dO_i/(i+1); dK_j = scale * sum_h sum_{i>=j} (dO_i.V_j - dO_i.O_i) Q_i/(i+1)
    D, L, Hq, Hkv = 8, 29, 4, 2
    G = Hq // Hkv
    cu, hq, hkv, q, k, v, do = _rand_problem(4, [L], [Hq], [Hkv], D)
    K = k.reshape(L, Hkv, D)
    K[:] = K[0:1]
    scale = 0.3
    O, LSE = oracle.attn_fwd(q, k, v, cu, hq, hkv, D, scale)
    dQ, dK, dV = oracle.attn_bwd(q, k, v, do, cu, hq, hkv, D, scale)
    Q, V, dO = q.reshape(L, Hq, D), v.reshape(L, Hkv, D), do.reshape(L, Hq, D)
    O = O.reshape(L, Hq, D)
    cnt = np.arange(1, L + 1)[:, None]
    for h in range(Hq):
        g = h // G
        np.testing.assert_allclose(O[:, h], np.cumsum(V[:, g], axis=0) / cnt, rtol=1e-13, atol=1e-14)
        np.testing.assert_allclose(LSE[h * L:(h + 1) * L], scale * Q[:, h] @ K[0, g] + np.log(cnt[:, 0]), rtol=1e-13)
    np.testing.assert_allclose(dQ, 0, atol=1e-13)
    edV = np.zeros((L, Hkv, D))
    edK = np.zeros((L, Hkv, D))
    for h in range(Hq):
        g = h // G
        Oh = np.cumsum(V[:, g], axis=0) / cnt
        for j in range(L):
            for i in range(j, L):
                edV[j, g] += dO[i, h] / (i + 1)
                edK[j, g] += scale * (dO[i, h] @ V[j, g] - dO[i, h] @ Oh[i]) * Q[i, h] / (i + 1)
    np.testing.assert_allclose(dV.reshape(L, Hkv, D), edV, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(dK.reshape(L, Hkv, D), edK, rtol=1e-12, atol=1e-13)


def test_gradient_identities():
    # softmax is invariant to a common shift of the keys  -> sum_j dK_j = 0
    # rows of P sum to one                                -> sum_j dV_j = sum_{h in g} sum_i dO_i
    # O is linear in V                                    -> <dV_g, V_g> = sum_{h in g} <dO_h, O_h>
    # S is bilinear in (Q, K)                             -> sum_{h in g} <dQ_h, Q_h> = <dK_g, K_g>
    D = 16
    cu, hq, hkv, q, k, v, do = _rand_problem(5, [40, 7], [6, 4], [2, 4], D)
    scale = 0.25
    O, _ = oracle.attn_fwd(q, k, v, cu, hq, hkv, D, scale)
    dQ, dK, dV = oracle.attn_bwd(q, k, v, do, cu, hq, hkv, D, scale)
    for s, L, Q, K, V, dO, qo, kvo, lo in _seg_views(cu, hq, hkv, D, q, k, v, do):
        G = hq[s] // hkv[s]
        Os = O[qo:qo + Q.size].reshape(Q.shape)
        dQs = dQ[qo:qo + Q.size].reshape(Q.shape)
        dKs = dK[kvo:kvo + K.size].reshape(K.shape)
        dVs = dV[kvo:kvo + K.size].reshape(K.shape)
        for g in range(hkv[s]):
            hs = slice(g * G, (g + 1) * G)
            np.testing.assert_allclose(dKs[:, g].sum(axis=0), 0, atol=1e-12)
            np.testing.assert_allclose(dVs[:, g].sum(axis=0), dO[:, hs].sum(axis=(0, 1)), rtol=1e-12, atol=1e-12)
            assert abs((dVs[:, g] * V[:, g]).sum() - (dO[:, hs] * Os[:, hs]).sum()) < 1e-11
            assert abs((dQs[:, hs] * Q[:, hs]).sum() - (dKs[:, g] * K[:, g]).sum()) < 1e-11


def test_output_is_convex_combination_of_visible_values():
    D = 8
    cu, hq, hkv, q, k, v, do = _rand_problem(6, [33], [2], [1], D)
    O, _ = oracle.attn_fwd(q, k, v, cu, hq, hkv, D, 0.9)
    O = O.reshape(33, 2, D)
    V = v.reshape(33, 1, D)
    for i in range(33):
        lo, hi = V[: i + 1, 0].min(axis=0), V[: i + 1, 0].max(axis=0)
        assert np.all(O[i] >= lo - 1e-13) and np.all(O[i] <= hi + 1e-13)


def test_packing_order_invariance_is_bitwise():
    D = 8
    lengths, hq, hkv = [13, 5, 21], [4, 2, 4], [2, 2, 1]
    cu, hq, hkv, q, k, v, do = _rand_problem(7, lengths, hq, hkv, D)
    scale = 0.4
    O, LSE = oracle.attn_fwd(q, k, v, cu, hq, hkv, D, scale)
    dQ, dK, dV = oracle.attn_bwd(q, k, v, do, cu, hq, hkv, D, scale)
    segs = list(_seg_views(cu, hq, hkv, D, q, k, v, do))
    perm = [2, 0, 1]
    pl = [lengths[p] for p in perm]
    pcu = np.concatenate([[0], np.cumsum(pl)]).astype(np.int32)
    phq, phkv = hq[perm], hkv[perm]
    pq = np.concatenate([segs[p][2].ravel() for p in perm])
    pk = np.concatenate([segs[p][3].ravel() for p in perm])
    pv = np.concatenate([segs[p][4].ravel() for p in perm])
    pdo = np.concatenate([segs[p][5].ravel() for p in perm])
    pO, pLSE = oracle.attn_fwd(pq, pk, pv, pcu, phq, phkv, D, scale)
    pdQ, pdK, pdV = oracle.attn_bwd(pq, pk, pv, pdo, pcu, phq, phkv, D, scale)
    psegs = list(_seg_views(pcu, phq, phkv, D, pq, pk, pv, pdo))
    for new_pos, p in enumerate(perm):
        _, L, Q, K, *_rest = segs[p]
        qo, kvo, lo = segs[p][6], segs[p][7], segs[p][8]
        nqo, nkvo, nlo = psegs[new_pos][6], psegs[new_pos][7], psegs[new_pos][8]
        np.testing.assert_array_equal(O[qo:qo + Q.size], pO[nqo:nqo + Q.size])
        np.testing.assert_array_equal(dQ[qo:qo + Q.size], pdQ[nqo:nqo + Q.size])
        np.testing.assert_array_equal(dK[kvo:kvo + K.size], pdK[nkvo:nkvo + K.size])
        np.testing.assert_array_equal(dV[kvo:kvo + K.size], pdV[nkvo:nkvo + K.size])
        np.testing.assert_array_equal(LSE[lo:lo + L * hq[p]], pLSE[nlo:nlo + L * hq[p]])
    # a segment alone gives the same result as the segment packed with others
    s1 = segs[1]
    aO, _ = oracle.attn_fwd(s1[2].ravel(), s1[3].ravel(), s1[4].ravel(), [0, lengths[1]], [hq[1]], [hkv[1]], D, scale)
    np.testing.assert_array_equal(aO, O[s1[6]:s1[6] + s1[2].size])


def test_backward_is_linear_in_dO():
    D = 8
    cu, hq, hkv, q, k, v, do1 = _rand_problem(8, [19, 4], [4, 4], [2, 2], D)
    do2 = np.random.default_rng(81).standard_normal(do1.size)
    a = 1.75
    g1 = oracle.attn_bwd(q, k, v, do1, cu, hq, hkv, D, 0.35)
    g2 = oracle.attn_bwd(q, k, v, do2, cu, hq, hkv, D, 0.35)
    g3 = oracle.attn_bwd(q, k, v, a * do1 + do2, cu, hq, hkv, D, 0.35)
    for x, y, z in zip(g1, g2, g3):
        np.testing.assert_allclose(z, a * x + y, rtol=1e-11, atol=1e-12)


def test_reduces_to_torch_sdpa_and_autograd():
    # single segment, and GQA expressed by repeating KV heads: the textbook causal SDPA
    torch = pytest.importorskip("torch")
    D, L, Hq, Hkv = 16, 45, 6, 2
    G = Hq // Hkv
    cu, hq, hkv, q, k, v, do = _rand_problem(9, [L], [Hq], [Hkv], D)
    scale = 1.0 / np.sqrt(D)
    O, _ = oracle.attn_fwd(q, k, v, cu, hq, hkv, D, scale)
    dQ, dK, dV = oracle.attn_bwd(q, k, v, do, cu, hq, hkv, D, scale)
    tq = torch.tensor(q.reshape(L, Hq, D)).permute(1, 0, 2).clone().requires_grad_(True)
    tk = torch.tensor(k.reshape(L, Hkv, D)).permute(1, 0, 2).clone().requires_grad_(True)
    tv = torch.tensor(v.reshape(L, Hkv, D)).permute(1, 0, 2).clone().requires_grad_(True)
    tO = torch.nn.functional.scaled_dot_product_attention(
        tq[None], tk.repeat_interleave(G, 0)[None], tv.repeat_interleave(G, 0)[None], is_causal=True, scale=scale)[0]
    tO.backward(torch.tensor(do.reshape(L, Hq, D)).permute(1, 0, 2))
    np.testing.assert_allclose(O.reshape(L, Hq, D), tO.detach().permute(1, 0, 2).numpy(), rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(dQ.reshape(L, Hq, D), tq.grad.permute(1, 0, 2).numpy(), rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(dK.reshape(L, Hkv, D), tk.grad.permute(1, 0, 2).numpy(), rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(dV.reshape(L, Hkv, D), tv.grad.permute(1, 0, 2).numpy(), rtol=1e-9, atol=1e-11)


def test_sampled_modes_agree_with_full_and_are_pinned_by_it():
    D = 8
    lengths, hq_, hkv_ = [31, 0, 12], [4, 4, 6], [2, 2, 3]
    cu, hq, hkv, q, k, v, do = _rand_problem(10, lengths, hq_, hkv_, D)
    scale = 0.33
    O, LSE = oracle.attn_fwd(q, k, v, cu, hq, hkv, D, scale)
    dQ, dK, dV = oracle.attn_bwd(q, k, v, do, cu, hq, hkv, D, scale)
    segs = {s[0]: s for s in _seg_views(cu, hq, hkv, D, q, k, v, do)}
    rows = [(0, 0, 0), (0, 3, 30), (0, 1, 17), (2, 5, 11), (2, 0, 0), (2, 2, 6)]
    sO, sLSE, sdQ = oracle.attn_rows(q, k, v, do, cu, hq, hkv, D, scale, rows)
    for t, (s, h, i) in enumerate(rows):
        qo, lo, L = segs[s][6], segs[s][8], segs[s][1]
        off = qo + (i * hq[s] + h) * D
        np.testing.assert_allclose(sO[t], O[off:off + D], rtol=1e-13, atol=1e-14)
        np.testing.assert_allclose(sdQ[t], dQ[off:off + D], rtol=1e-12, atol=1e-13)
        assert abs(sLSE[t] - LSE[lo + h * L + i]) < 1e-13
    cols = [(0, 0, 30), (0, 1, 25), (0, 1, 0), (2, 2, 11), (2, 0, 3)]
    sdK, sdV = oracle.attn_cols(q, k, v, do, cu, hq, hkv, D, scale, cols)
    for t, (s, g, j) in enumerate(cols):
        off = segs[s][7] + (j * hkv[s] + g) * D
        np.testing.assert_allclose(sdK[t], dK[off:off + D], rtol=1e-12, atol=1e-13)
        np.testing.assert_allclose(sdV[t], dV[off:off + D], rtol=1e-12, atol=1e-13)
    # row-subset backward equals the full backward when dO vanishes off the subset
    active = [(0, 2), (0, 30), (2, 5), (2, 0)]
    do_sparse = np.zeros_like(do)
    for s, i in active:
        qo = segs[s][6]
        do_sparse[qo + i * hq[s] * D: qo + (i + 1) * hq[s] * D] = do[qo + i * hq[s] * D: qo + (i + 1) * hq[s] * D]
    full = oracle.attn_bwd(q, k, v, do_sparse, cu, hq, hkv, D, scale)
    sub = oracle.attn_bwd(q, k, v, do_sparse, cu, hq, hkv, D, scale, rows=active)
    for a, b in zip(full, sub):
        np.testing.assert_allclose(a, b, rtol=1e-13, atol=1e-15)
    # and dQ is exactly zero off the active rows
    dq_full = full[0]
    mask = np.ones(dq_full.size, bool)
    for s, i in active:
        qo = segs[s][6]
        mask[qo + i * hq[s] * D: qo + (i + 1) * hq[s] * D] = False
    assert np.all(dq_full[mask] == 0)


def test_bf16_inputs_are_widened_exactly():
    # bf16 bit patterns: 0x3F80 = 1, 0xC000 = -2, 0x3E80 = 0.25, 0x4049 = 3.140625
    D = 2
    q = np.array([0x3F80, 0xC000], np.uint16)
    k = np.array([0x3E80, 0x4049], np.uint16)
    v = np.array([0x4049, 0xC000], np.uint16)
    O, LSE = oracle.attn_fwd(q, k, v, [0, 1], [1], [1], D, 2.0)
    np.testing.assert_array_equal(O, [3.140625, -2.0])
    assert LSE[0] == 2.0 * (1 * 0.25 + (-2.0) * 3.140625)


def test_hand_computed_fixture():
    """tests/golden/attention_tiny.txt: a 2-token, 1-head, D=1 case worked out by hand from the definition."""
    path = os.path.join(os.path.dirname(__file__), "golden", "attention_tiny.txt")
    vals = {}
    for line in open(path):
        line = line.split("#")[0].strip()
        if line:
            key, rest = line.split("=")
            vals[key.strip()] = np.array([float(x) for x in rest.split()])
    cu, hq, hkv = [0, 2], [1], [1]
    O, LSE = oracle.attn_fwd(vals["q"], vals["k"], vals["v"], cu, hq, hkv, 1, float(vals["scale"][0]))
    dQ, dK, dV = oracle.attn_bwd(vals["q"], vals["k"], vals["v"], vals["dO"], cu, hq, hkv, 1, float(vals["scale"][0]))
    np.testing.assert_allclose(O, vals["O"], rtol=1e-14)
    np.testing.assert_allclose(LSE, vals["LSE"], rtol=1e-14)
    np.testing.assert_allclose(dQ, vals["dQ"], rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(dK, vals["dK"], rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(dV, vals["dV"], rtol=1e-13, atol=1e-15)
