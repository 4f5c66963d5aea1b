"""Pins of the CPU oracle against things other than itself (CPU only).

Each test fixes some part of the oracle to what the paper's definitions and plain
mathematics determine: a dense-then-mask brute force written with numpy array
operations (no grouping, no permutation), reductions to a dense MLP and to the
unrestricted layer of Section 2, routing invariants, gate normalisation, and
closed forms of the importance score, Eq. (1).
"""
import math

import numpy as np
import pytest

import oracle
from paper_2308_15030_b200 import inputs as I


# ------------------------------------------------------------------ independent brute force
def _softmax_rows(l):
    m = np.max(l, axis=1, keepdims=True)
    e = np.exp(l - m)
    return e / e.sum(axis=1, keepdims=True)


def brute_force_layer(x, Wr, experts, resident, k, act, renorm):
    """Dense-then-mask evaluation: every expert on every token, then a dense gate matrix.

    experts: list over ALL E experts of (w_in [nin,f,d], w_out [d,f]);
    resident: iterable of expert ids allowed by Masked Gating (Fig. 4).
    Returns (out [T,d], Gdense [T,E]).
    """
    x = x.astype(np.float64)
    T, d = x.shape
    E = Wr.shape[0]
    logits = x @ Wr.astype(np.float64).T
    masked = np.full_like(logits, -np.inf)
    res = sorted(int(e) for e in resident)
    masked[:, res] = logits[:, res]
    p = _softmax_rows(masked)                      # zero outside the resident set
    order = np.argsort(-masked, axis=1, kind="stable")[:, :k]   # ties -> lowest index
    G = np.zeros((T, E))
    for t in range(T):
        sel = order[t]
        w = p[t, sel]
        if renorm:
            w = w / w.sum()
        G[t, sel] = w
    dense = np.zeros((E, T, d))
    for e in res:
        w_in, w_out = experts[e]
        a = x @ w_in[0].astype(np.float64).T
        if act == I.ACT_SWIGLU:
            b = x @ w_in[1].astype(np.float64).T
            h = a / (1.0 + np.exp(-a)) * b
        else:
            h = np.maximum(a, 0.0)
        dense[e] = h @ w_out.astype(np.float64).T
    out = np.einsum("te,etd->td", G, dense)
    return out, G


def _tiny(seed, T, d, f, E, k, K, act, renorm, dtype=I.F32):
    cfg = I.LayerConfig("tiny", dtype, T=T, d=d, f=f, E=E, k=k, K=K, act=act, renorm=renorm,
                        seed=seed)
    rng = np.random.default_rng(seed + 100)
    Wr = I.make_router(cfg)
    x = I.make_tokens(cfg, Wr)
    experts = [I.make_expert(cfg, e) for e in range(E)]
    # make the experts big enough that outputs are O(1)
    experts = [(w_in * 25, w_out * 25) for (w_in, w_out) in experts]
    enorm = (1.0 + rng.random(E)).astype(np.float32)
    s2e = rng.permutation(E)[:K].astype(np.int32)
    P = K + 2
    phys = rng.permutation(P)[:K].astype(np.int32)
    a_in = np.zeros((P, cfg.nin, f, d), np.float32)
    a_out = np.zeros((P, d, f), np.float32)
    for s, e in enumerate(s2e):
        a_in[phys[s]], a_out[phys[s]] = experts[e]
    return cfg, x, Wr, experts, enorm, s2e, phys, a_in, a_out


CASES = [
    (0, 16, 24, 32, 8, 1, 4, I.ACT_RELU, 0),
    (1, 13, 32, 20, 8, 2, 4, I.ACT_SWIGLU, 1),
    (2, 16, 16, 32, 6, 2, 3, I.ACT_RELU, 0),
    (3, 11, 8, 12, 5, 1, 1, I.ACT_SWIGLU, 0),
    (4, 16, 32, 32, 8, 2, 8, I.ACT_SWIGLU, 1),
    (5, 9, 16, 16, 7, 3, 5, I.ACT_RELU, 1),
]


@pytest.mark.parametrize("case", CASES)
def test_dense_then_mask_brute_force(case):
    seed, T, d, f, E, k, K, act, renorm = case
    cfg, x, Wr, experts, enorm, s2e, phys, a_in, a_out = _tiny(seed, T, d, f, E, k, K, act, renorm)
    r = oracle.forward(x, Wr, enorm, s2e, a_in, a_out, k=k, act=act, renorm=renorm, phys_slot=phys)
    ref, G = brute_force_layer(x, Wr, experts, s2e, k, act, renorm)
    assert np.max(np.abs(r["out"] - ref)) <= 1e-12 * max(1.0, np.max(np.abs(ref)))
    # the oracle's sparse (midx, mgate) must be the dense gate matrix
    G2 = np.zeros_like(G)
    for t in range(T):
        for j in range(k):
            G2[t, r["midx"][t, j]] += r["mgate"][t, j]
    assert np.max(np.abs(G - G2)) <= 1e-14


@pytest.mark.parametrize("act,k,renorm", [(I.ACT_RELU, 1, 0), (I.ACT_SWIGLU, 2, 1)])
def test_full_budget_equals_unrestricted_layer(act, k, renorm):
    """K = E: the Virtual-Expert layer is the off-the-shelf layer, y = G(x)_i E_i(x) (Section 2)."""
    seed, T, d, f, E = 7, 16, 16, 24, 6
    cfg, x, Wr, experts, enorm, s2e, phys, a_in, a_out = _tiny(seed, T, d, f, E, k, E, act, renorm)
    r = oracle.forward(x, Wr, enorm, s2e, a_in, a_out, k=k, act=act, renorm=renorm, phys_slot=phys)
    ref, _ = brute_force_layer(x, Wr, experts, range(E), k, act, renorm)
    assert np.max(np.abs(r["out"] - ref)) <= 1e-12 * np.max(np.abs(ref))
    # with every expert resident the masked and the unmasked gate coincide
    assert np.array_equal(r["uidx"], r["midx"])
    assert np.max(np.abs(r["ugate"] - r["mgate"])) == 0.0


@pytest.mark.parametrize("case", CASES[:4])
def test_expert_hidden_is_the_inner_half_of_the_expert(case):
    """oracle.expert_hidden against numpy: row p is act(W_in x) of pair p's token under pair p's
    expert (dense evaluation of every resident expert, then picked), and W_out applied to it
    reproduces the expert outputs the layer's own evaluation returns."""
    seed, T, d, f, E, k, K, act, renorm = case
    cfg, x, Wr, experts, enorm, s2e, phys, a_in, a_out = _tiny(seed, T, d, f, E, k, K, act, renorm)
    r = oracle.forward(x, Wr, enorm, s2e, a_in, a_out, k=k, act=act, renorm=renorm, phys_slot=phys,
                       want_y=True)
    h = oracle.expert_hidden(x, r["slot"], phys, a_in, k=k, act=act)
    x64 = x.astype(np.float64)
    for t in range(T):
        for j in range(k):
            w_in, w_out = experts[r["midx"][t, j]]
            a = w_in[0].astype(np.float64) @ x64[t]
            ref = a / (1 + np.exp(-a)) * (w_in[1].astype(np.float64) @ x64[t]) if act == I.ACT_SWIGLU \
                else np.maximum(a, 0)
            assert np.max(np.abs(h[t * k + j] - ref)) <= 1e-12 * max(1.0, np.max(np.abs(ref)))
            y = w_out.astype(np.float64) @ h[t * k + j]
            assert np.max(np.abs(y - r["y"][t * k + j])) <= 1e-12 * max(1.0, np.max(np.abs(y)))
    # a token subset leaves the other rows at zero and changes nothing else
    sub = np.array([1, 4, 7], np.int32)
    hs = oracle.expert_hidden(x, r["slot"], phys, a_in, k=k, act=act, token_subset=sub)
    rows = (sub[:, None] * k + np.arange(k)[None, :]).reshape(-1)
    assert np.array_equal(hs[rows], h[rows])
    mask = np.ones(T * k, bool); mask[rows] = False
    assert not hs[mask].any()


@pytest.mark.parametrize("act", [I.ACT_RELU, I.ACT_SWIGLU])
def test_single_expert_is_a_dense_mlp(act):
    """E = K = 1: gate is exactly 1 and the layer is W_out * act(W_in * x)."""
    cfg, x, Wr, experts, enorm, s2e, phys, a_in, a_out = _tiny(3, 12, 16, 24, 1, 1, 1, act, 0)
    r = oracle.forward(x, Wr, enorm, s2e, a_in, a_out, k=1, act=act, renorm=0, phys_slot=phys)
    assert np.all(r["mgate"] == 1.0) and np.all(r["ugate"] == 1.0)
    w_in, w_out = experts[0]
    x64 = x.astype(np.float64)
    a = x64 @ w_in[0].astype(np.float64).T
    if act == I.ACT_SWIGLU:
        h = a / (1 + np.exp(-a)) * (x64 @ w_in[1].astype(np.float64).T)
    else:
        h = np.maximum(a, 0)
    ref = h @ w_out.astype(np.float64).T
    assert np.max(np.abs(r["out"] - ref)) <= 1e-12 * np.max(np.abs(ref))


def test_hand_worked_example():
    """Two tokens, three experts, worked by hand from y = G(x)_i E_i(x) and Eq. (1)."""
    x = np.array([[1, 2], [3, -1]], np.float32)
    Wr = np.array([[1, 0], [0, 1], [1, 1]], np.float32)      # logits: [1,2,3], [3,-1,2]
    s2e = np.array([2, 0], np.int32)                          # slot 0 -> expert 2, slot 1 -> expert 0
    a_in = np.zeros((2, 1, 2, 2), np.float32)
    a_out = np.zeros((2, 2, 2), np.float32)
    a_in[0, 0] = [[1, -1], [0.5, 0.5]]; a_out[0] = [[1, 2], [0, -1]]     # expert 2
    a_in[1, 0] = [[1, 0], [0, 1]];      a_out[1] = [[2, 0], [1, 1]]      # expert 0
    enorm = np.array([1, 2, 3], np.float32)
    r = oracle.forward(x, Wr, enorm, s2e, a_in, a_out, k=1, act=I.ACT_RELU, renorm=0)
    assert r["uidx"].ravel().tolist() == [2, 0]
    assert r["midx"].ravel().tolist() == [2, 0]
    assert r["slot"].ravel().tolist() == [0, 1]
    assert r["count"].tolist() == [1, 1] and r["offset"].tolist() == [0, 1, 2]
    ug0 = 1 / (1 + math.exp(-1) + math.exp(-2)); ug1 = 1 / (1 + math.exp(-4) + math.exp(-1))
    mg0 = 1 / (1 + math.exp(-2)); mg1 = 1 / (1 + math.exp(-1))
    assert np.allclose(r["ugate"].ravel(), [ug0, ug1], rtol=0, atol=1e-15)
    assert np.allclose(r["mgate"].ravel(), [mg0, mg1], rtol=0, atol=1e-15)
    # expert 2 on [1,2]: relu([-1,1.5]) = [0,1.5] -> [3,-1.5]; expert 0 on [3,-1]: relu -> [3,0] -> [6,3]
    ref = np.array([[3 * mg0, -1.5 * mg0], [6 * mg1, 3 * mg1]])
    assert np.allclose(r["out"], ref, rtol=0, atol=1e-14)
    imp = np.array([math.sqrt(10) * ug1 * 1, 0.0, math.sqrt(5) * ug0 * 3])
    assert np.allclose(r["imp"], imp, rtol=0, atol=1e-14)


# ------------------------------------------------------------------ routing invariants
@pytest.mark.parametrize("k,renorm", [(1, 0), (2, 1), (2, 0)])
def test_routing_invariants(k, renorm):
    rng = np.random.default_rng(5)
    T, E, K = 300, 16, 6
    logits = rng.normal(size=(T, E)).astype(np.float32)
    logits[10:20] = 0.25                      # rows of exact ties
    logits[30, :] = np.float32(1.0)
    s2e = rng.permutation(E)[:K].astype(np.int32)
    e2s = oracle.invert_slot_table(s2e, E)
    allowed = (e2s >= 0).astype(np.int32)
    uidx, ugate = oracle.gate(logits, k, renorm)
    midx, mgate = oracle.gate(logits, k, renorm, allowed)
    # masked selections are resident; if the unmasked top-1 is resident the masked top-1 is the same
    assert np.all(allowed[midx] == 1)
    same = allowed[uidx[:, 0]] == 1
    assert np.array_equal(midx[same, 0], uidx[same, 0])
    # k distinct experts per token, ordered by descending logit
    for t in range(T):
        assert len(set(midx[t])) == k and len(set(uidx[t])) == k
        assert np.all(np.diff(logits[t, uidx[t]]) <= 0)
        assert np.all(np.diff(logits[t, midx[t]]) <= 0)
    # all-equal logits: lowest (resident) index first
    assert uidx[30, 0] == 0 and midx[30, 0] == np.flatnonzero(allowed)[0]
    assert uidx[12, 0] == 0
    slot = e2s[midx]
    count, offset, perm, inv = oracle.permute(slot, K)
    assert count.sum() == T * k and offset[0] == 0 and offset[-1] == T * k
    assert np.array_equal(np.diff(offset), count)
    assert np.array_equal(np.bincount(slot.ravel(), minlength=K), count)
    assert np.array_equal(np.sort(perm), np.arange(T * k))          # a permutation
    assert np.array_equal(inv[perm], np.arange(T * k))              # inv o perm = id
    flat_slot = slot.ravel()
    for s in range(K):
        seg = perm[offset[s]:offset[s + 1]]
        assert np.all(flat_slot[seg] == s)
        assert np.all(np.diff(seg) > 0)                              # ascending flat index
    # equals numpy's stable sort by slot
    assert np.array_equal(perm, np.argsort(flat_slot, kind="stable"))


def test_gate_normalisation_and_uniform_logits():
    rng = np.random.default_rng(9)
    T, E = 64, 12
    logits = rng.normal(scale=3.0, size=(T, E)).astype(np.float32)
    allowed = np.zeros(E, np.int32); allowed[[1, 4, 5, 9, 11]] = 1
    # k = |R| without renormalisation lists the whole masked softmax: sums to one
    idx, g = oracle.gate(logits, 5, 0, allowed)
    assert np.allclose(g.sum(axis=1), 1.0, rtol=0, atol=1e-14)
    # and it is the softmax over the resident logits
    p = _softmax_rows(logits[:, [1, 4, 5, 9, 11]].astype(np.float64))
    assert np.allclose(np.sort(g, axis=1), np.sort(p, axis=1), rtol=0, atol=1e-15)
    # top-2 renormalised gates sum to one
    _, g2 = oracle.gate(logits, 2, 1, allowed)
    assert np.allclose(g2.sum(axis=1), 1.0, rtol=0, atol=1e-15)
    # k = 1 value is the softmax probability of the argmax
    i1, g1 = oracle.gate(logits, 1, 0)
    pf = _softmax_rows(logits.astype(np.float64))
    assert np.array_equal(i1[:, 0], np.argmax(logits, axis=1))
    assert np.allclose(g1[:, 0], pf.max(axis=1), rtol=0, atol=1e-15)
    # constant logits: p = 1/|R|
    _, gc = oracle.gate(np.full((3, E), 2.5, np.float32), 1, 0, allowed)
    assert np.allclose(gc, 1.0 / 5, rtol=0, atol=1e-16)
    with pytest.raises(ValueError):
        oracle.gate(logits, 6, 0, allowed)


def test_mask_after_softmax_differs_only_in_value():
    """Fig. 4 reading: masking before the softmax keeps the argmax over R and renormalises."""
    rng = np.random.default_rng(2)
    logits = rng.normal(size=(50, 8)).astype(np.float32)
    allowed = np.array([0, 1, 1, 0, 0, 1, 0, 0], np.int32)
    midx, mgate = oracle.gate(logits, 1, 0, allowed)
    pf = _softmax_rows(logits.astype(np.float64))
    pm = pf * allowed
    assert np.array_equal(midx[:, 0], np.argmax(pm, axis=1))
    assert np.allclose(mgate[:, 0], pm.max(axis=1) / pm.sum(axis=1), rtol=0, atol=1e-15)


# ------------------------------------------------------------------ output properties
def test_token_order_invariance_and_zero_rows():
    cfg, x, Wr, experts, enorm, s2e, phys, a_in, a_out = _tiny(11, 16, 16, 24, 8, 2, 4,
                                                                I.ACT_SWIGLU, 1)
    x = x.copy(); x[5] = 0.0
    r = oracle.forward(x, Wr, enorm, s2e, a_in, a_out, k=2, act=I.ACT_SWIGLU, renorm=1, phys_slot=phys)
    assert np.all(r["out"][5] == 0.0)                                # no biases
    p = np.random.default_rng(0).permutation(16)
    r2 = oracle.forward(x[p], Wr, enorm, s2e, a_in, a_out, k=2, act=I.ACT_SWIGLU, renorm=1,
                        phys_slot=phys)
    assert np.array_equal(r2["out"], r["out"][p])                   # exact: rows are independent
    assert np.allclose(r2["imp"], r["imp"], rtol=1e-14)


def test_token_subset_matches_full():
    cfg, x, Wr, experts, enorm, s2e, phys, a_in, a_out = _tiny(12, 16, 16, 24, 8, 2, 4, I.ACT_RELU, 0)
    r = oracle.forward(x, Wr, enorm, s2e, a_in, a_out, k=2, act=I.ACT_RELU, renorm=0, phys_slot=phys)
    sub = np.array([3, 7, 8], np.int32)
    r2 = oracle.forward(x, Wr, enorm, s2e, a_in, a_out, k=2, act=I.ACT_RELU, renorm=0,
                        phys_slot=phys, token_subset=sub)
    assert np.array_equal(r2["out"][sub], r["out"][sub])
    assert np.array_equal(r2["perm"], r["perm"])


def test_external_logits_replace_router():
    cfg, x, Wr, experts, enorm, s2e, phys, a_in, a_out = _tiny(13, 16, 16, 24, 8, 1, 4, I.ACT_RELU, 0)
    ext = np.random.default_rng(1).normal(size=(16, 8)).astype(np.float32)
    r = oracle.forward(x, Wr, enorm, s2e, a_in, a_out, k=1, act=I.ACT_RELU, renorm=0,
                       phys_slot=phys, ext_logits=ext)
    assert np.array_equal(r["logits"], ext.astype(np.float64))
    assert np.array_equal(r["uidx"][:, 0], np.argmax(ext, axis=1))


def test_logits_match_matmul():
    rng = np.random.default_rng(3)
    x = rng.normal(size=(33, 70)).astype(np.float32)
    Wr = rng.normal(size=(9, 70)).astype(np.float32)
    ref = x.astype(np.float64) @ Wr.astype(np.float64).T
    assert np.allclose(oracle.logits(x, Wr), ref, rtol=0, atol=1e-12)


# ------------------------------------------------------------------ Eq. (1) closed forms
def test_importance_closed_forms():
    rng = np.random.default_rng(4)
    T, d, E = 40, 24, 6
    x = rng.normal(size=(T, d))
    x = (x / np.linalg.norm(x, axis=1, keepdims=True)).astype(np.float32)   # ~unit norm
    xn = np.linalg.norm(x.astype(np.float64), axis=1)
    ones = np.ones(E, np.float32)
    logits = rng.normal(size=(T, E)).astype(np.float32)
    # k = 2 renormalised, enorm = 1: sum_e imp = sum_t ||x_t|| * (G_0 + G_1) = sum_t ||x_t||
    uidx, ugate = oracle.gate(logits, 2, 1)
    imp = oracle.importance(x, uidx, ugate, ones)
    assert abs(imp.sum() - xn.sum()) <= 1e-12
    # constant logits, k = 1: everything lands on expert 0 with gate 1/E
    uidx, ugate = oracle.gate(np.zeros((T, E), np.float32), 1, 0)
    imp = oracle.importance(x, uidx, ugate, ones)
    assert abs(imp[0] - xn.sum() / E) <= 1e-12 and np.all(imp[1:] == 0)
    # scaling x by alpha (fixed routing) scales importance by |alpha|; enorm enters linearly
    uidx, ugate = oracle.gate(logits, 1, 0)
    en = (1 + rng.random(E)).astype(np.float32)
    a = oracle.importance(x, uidx, ugate, en)
    b = oracle.importance((-4.0 * x).astype(np.float32), uidx, ugate, en)
    assert np.allclose(b, 4.0 * a, rtol=1e-14)
    c = oracle.importance(x, uidx, ugate, ones)
    assert np.allclose(a, c * en.astype(np.float64), rtol=1e-14)
    # additive over calls
    h = T // 2
    a1 = oracle.importance(x[:h], uidx[:h], ugate[:h], en)
    a2 = oracle.importance(x[h:], uidx[h:], ugate[h:], en, imp=a1)
    assert np.allclose(a2, a, rtol=1e-13)
    # direct evaluation of Eq. (1) with numpy
    ref = np.zeros(E)
    np.add.at(ref, uidx[:, 0], xn * ugate[:, 0] * en[uidx[:, 0]].astype(np.float64))
    assert np.allclose(a, ref, rtol=1e-14)
    # Eq. (1) is not the token count ("Simple scheduling" ablation)
    cnt = oracle.importance_count(uidx, E)
    assert np.array_equal(cnt, np.bincount(uidx[:, 0], minlength=E).astype(np.float64))


def test_importance_uses_unmasked_routing():
    cfg, x, Wr, experts, enorm, s2e, phys, a_in, a_out = _tiny(21, 16, 16, 24, 8, 1, 2, I.ACT_RELU, 0)
    r = oracle.forward(x, Wr, enorm, s2e, a_in, a_out, k=1, act=I.ACT_RELU, renorm=0, phys_slot=phys)
    absent = [e for e in range(8) if e not in set(s2e.tolist())]
    assert any(r["imp"][e] > 0 for e in absent)       # absent experts can still earn importance
    ref = oracle.importance(x, r["uidx"], r["ugate"], enorm)
    assert np.array_equal(ref, r["imp"])


def test_topk_importance_ties_lowest_index():
    imp = np.array([1.0, 5.0, 5.0, 0.5, 7.0, 5.0])
    assert oracle.topk_importance(imp, 3).tolist() == [4, 1, 2]
    assert oracle.topk_importance(imp, 6).tolist() == [4, 1, 2, 5, 0, 3]
    assert oracle.topk_importance(np.zeros(4), 2).tolist() == [0, 1]


def test_bad_slot_table_rejected():
    with pytest.raises(ValueError):
        oracle.invert_slot_table([1, 1], 4)
    with pytest.raises(ValueError):
        oracle.invert_slot_table([0, 4], 4)
