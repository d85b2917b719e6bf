"""Pins for the oracle's routing (Algorithm 1): a hand-worked example with exact
fractions, brute force with separately written rank formulas, invariants and
closed forms.  None of these retypes the oracle's loops: the expected values come
from hand arithmetic, from counting definitions evaluated by brute force, or from
special cases with a known answer.
"""
import json
import os
from fractions import Fraction as Fr

import numpy as np
import pytest

from oracle import gshard_oracle as orc

# ---------------------------------------------------------------------------
# Hand-worked example: one group, S=5 tokens, E=3 experts, capacity C=2.
# Gate probabilities are chosen by hand; x_s = (ln p_s, tag) with wg = [I3; 0]
# makes softmax(x.wg) return exactly p_s.  Every number below was worked out by
# hand with exact fractions, following Algorithm 1 step by step:
#   top-2:   s0 (0,1)  s1 (0,2)  s2 (0,1)  s3 (1,2)  s4 (2,1)
#   w1,w2:   2/3,1/3   5/9,4/9   7/9,2/9   5/8,3/8   2/3,1/3
#   loop 1:  s0 e0@0 keep, s1 e0@1 keep, s2 e0@2 DROP (C=2), s3 e1@0, s4 e2@0
#            -> c = (3,1,1)
#   m = (2.1, 1.4, 1.5)/5 = (21/50, 7/25, 3/10)
#   l_aux = (1/3)(3/5*21/50 + 1/5*7/25 + 1/5*3/10) = 46/375
#   loop 2 (counter advances for every token), u = (.5,.95,.1,.2,.9):
#     s0 e1@1, 2/3>.5 keep          -> c1=2
#     s1 e2@1, 8/9>.95 false: skip  -> c2=2 (slot 1 of e2 stays empty)
#     s2 e1@2 >= C drop             -> c1=3
#     s3 e2@2 >= C drop             -> c2=3
#     s4 e1@3 drop (and 2/3>.9 false) -> c1=4
#   total = (3,4,3)
#   other reading (only passing tokens advance): s1 leaves c2=1, so s3 gets
#   e2@1 and is kept; s4 fails the test, c1 stays 3: total = (3,3,2).
# ---------------------------------------------------------------------------
P = np.array([[0.6, 0.3, 0.1], [0.5, 0.1, 0.4], [0.7, 0.2, 0.1], [0.2, 0.5, 0.3], [0.1, 0.3, 0.6]])
U = np.array([0.5, 0.95, 0.1, 0.2, 0.9], np.float32)
TAG = np.arange(1, 6, dtype=np.float64)


def _example_inputs():
    S, E, M, H = 5, 3, 4, 1
    x = np.zeros((1, S, M), np.float32)
    x[0, :, :3] = np.log(P)
    x[0, :, 3] = TAG
    wg = np.zeros((M, E), np.float32)
    wg[:3, :3] = np.eye(3)
    wi = np.zeros((E, M, H), np.float32)
    wi[:, 3, 0] = 1.0                      # h = tag
    wo = np.zeros((E, H, M), np.float32)
    for e in range(E):
        wo[e, 0, 3] = e + 1.0              # FFN_e(x)[3] = (e+1) * tag
    return x, wg, wi, wo, U.reshape(1, S)


GOLDEN = json.load(open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "alg1_worked_example.json")))


def _fr(v):
    return float(Fr(v))


def test_golden_file_matches_the_inputs_used_here():
    assert np.array_equal(np.array(GOLDEN["gate_probabilities"]), P)
    assert np.allclose(np.array(GOLDEN["u"], np.float32), U)
    assert GOLDEN["token_tag"] == TAG.astype(int).tolist()


def test_worked_example_default_reading():
    x, wg, wi, wo, u = _example_inputs()
    f = orc.forward(x, wg, wi, wo, u, C=GOLDEN["C"])
    g = GOLDEN["default_reading"]
    assert f.expert_idx[0].tolist() == GOLDEN["expert_idx"]
    assert f.slot[0].tolist() == g["slot"]
    w_exp = [[_fr(a), _fr(b)] for a, b in GOLDEN["weight_fractions"]]
    np.testing.assert_allclose(f.weight[0], np.array(w_exp, dtype=np.float64), rtol=1e-6)
    # flags: bit0 first kept, bit1 random test passed, bit2 second kept
    assert f.flags[0].tolist() == g["flags"]
    assert f.first_count[0].tolist() == GOLDEN["first_count"]
    assert f.total_count[0].tolist() == g["total_count"]
    np.testing.assert_allclose(f.m[0], [_fr(v) for v in GOLDEN["mean_gates_fractions"]], rtol=1e-6)
    assert f.l_aux == pytest.approx(_fr(GOLDEN["l_aux_fraction"]), rel=1e-6)
    assert f.l_aux_group[0] == pytest.approx(_fr(GOLDEN["l_aux_fraction"]), rel=1e-6)
    # slot_token [E,G,C]: e0 <- s0,s1 ; e1 <- s3,s0 ; e2 <- s4,empty
    assert f.slot_token[:, 0, :].tolist() == g["slot_token"]
    np.testing.assert_allclose(f.y[0, :, 3], [_fr(v) for v in g["y_tag_component_fractions"]], rtol=1e-6)
    assert np.all(f.y[0, :, :3] == 0.0)


def test_worked_example_other_reading():
    x, wg, wi, wo, u = _example_inputs()
    f = orc.forward(x, wg, wi, wo, u, C=GOLDEN["C"], variant_a=True)
    g = GOLDEN["other_reading"]
    assert f.slot[0].tolist() == g["slot"]
    assert f.total_count[0].tolist() == g["total_count"]
    assert f.first_count[0].tolist() == GOLDEN["first_count"]
    np.testing.assert_allclose(f.y[0, :, 3], [_fr(v) for v in g["y_tag_component_fractions"]], rtol=1e-6)
    assert f.l_aux == pytest.approx(_fr(GOLDEN["l_aux_fraction"]), rel=1e-6)


def test_tie_lowest_index_wins():
    # p = (0.4, 0.4, 0.2): both picks tie-break to the lower index; w1 = w2 = 1/2 and
    # 2*w2 = 1 > u for every u in [0,1).  A second row ties the 2nd and 3rd gates.
    p = np.array([[0.4, 0.4, 0.2], [0.5, 0.25, 0.25], [0.2, 0.4, 0.4]])
    e1, e2, g1, g2, g3 = orc.top2(p)
    assert e1.tolist() == [0, 0, 1] and e2.tolist() == [1, 1, 2]
    assert g1.tolist() == [0.4, 0.5, 0.4] and g2.tolist() == [0.4, 0.25, 0.4]
    assert g3.tolist() == [0.2, 0.25, 0.2]
    u = np.array([0.0, 0.5, 0.999999], np.float32)
    r = orc.capacity(3, 3, e1, e2, g1, g2, u, m=np.ones(3) / 3)
    assert r.weight[0].tolist() == [0.5, 0.5]
    assert (r.flags[0] & 2) and (r.flags[2] & 2)


# ---------------------------------------------------------------------------
# Brute force on tiny inputs.  Expected values are computed from the counting
# definitions ("how many earlier tokens picked this expert"), evaluated with
# O(S^2) scans, not with running counters.
# ---------------------------------------------------------------------------
def _brute(S, E, C, e1, e2, g1, g2, u, variant_a):
    w1 = [g1[s] / (g1[s] + g2[s]) for s in range(S)]
    w2 = [g2[s] / (g1[s] + g2[s]) for s in range(S)]
    passed = [2.0 * w2[s] > float(u[s]) for s in range(S)]
    n_first = [sum(1 for t in range(S) if e1[t] == e) for e in range(E)]
    slot = np.full((S, 2), -1, np.int64)
    for s in range(S):
        rank1 = sum(1 for t in range(s) if e1[t] == e1[s])
        if rank1 < C:
            slot[s, 0] = rank1
        earlier = [t for t in range(s) if e2[t] == e2[s] and (passed[t] or not variant_a)]
        rank2 = n_first[e2[s]] + len(earlier)
        if rank2 < C and passed[s]:
            slot[s, 1] = rank2
    total = [n_first[e] + sum(1 for t in range(S) if e2[t] == e and (passed[t] or not variant_a))
             for e in range(E)]
    return slot, passed, n_first, total, w1, w2


@pytest.mark.parametrize("variant_a", [False, True])
def test_capacity_brute_force(variant_a):
    rng = np.random.default_rng(7)
    for trial in range(400):
        S = int(rng.integers(1, 9))
        E = int(rng.integers(2, 5))
        C = int(rng.integers(1, 4))
        p = rng.dirichlet(np.ones(E) * 0.7, size=S)
        order = np.argsort(-p, axis=1, kind="stable")        # brute-force top-2 by sorting
        e1, e2 = order[:, 0], order[:, 1]
        g1, g2 = p[np.arange(S), e1], p[np.arange(S), e2]
        o1, o2, og1, og2, _ = orc.top2(p)
        assert o1.tolist() == e1.tolist() and o2.tolist() == e2.tolist()
        assert og1.tolist() == g1.tolist() and og2.tolist() == g2.tolist()
        u = rng.random(S).astype(np.float32)
        m = p.mean(axis=0)
        r = orc.capacity(E, C, e1, e2, g1, g2, u, m, variant_a=variant_a)
        slot, passed, n_first, total, w1, w2 = _brute(S, E, C, e1, e2, g1, g2, u, variant_a)
        assert r.slot.tolist() == slot.tolist(), (trial, S, E, C)
        assert ((r.flags & 2) != 0).tolist() == passed
        assert ((r.flags & 1) != 0).tolist() == (slot[:, 0] >= 0).tolist()
        assert ((r.flags & 4) != 0).tolist() == (slot[:, 1] >= 0).tolist()
        assert r.first_count.tolist() == n_first
        assert r.total_count.tolist() == total
        np.testing.assert_allclose(r.weight[:, 0], w1, rtol=1e-14)
        np.testing.assert_allclose(r.weight[:, 1], w2, rtol=1e-14)
        l_aux = sum(Fr(n_first[e], S) * Fr(float(m[e])) for e in range(E)) / E   # exact rationals
        assert r.l_aux == pytest.approx(float(l_aux), rel=1e-12)


def test_pass_override_replays_forced_decisions():
    rng = np.random.default_rng(3)
    S, E, C = 64, 4, 12
    p = rng.dirichlet(np.ones(E), size=S)
    e1, e2, g1, g2, _ = orc.top2(p)
    u = rng.random(S).astype(np.float32)
    base = orc.capacity(E, C, e1, e2, g1, g2, u, p.mean(0))
    natural = ((base.flags & 2) != 0).astype(np.int8)
    same = orc.capacity(E, C, e1, e2, g1, g2, u, p.mean(0), pass_override=natural)
    assert same.slot.tolist() == base.slot.tolist()
    forced = np.full(S, -1, np.int8)
    forced[10] = 1 - natural[10]
    flipped = orc.capacity(E, C, e1, e2, g1, g2, u, p.mean(0), pass_override=forced)
    assert bool(flipped.flags[10] & 2) == bool(forced[10])


# ---------------------------------------------------------------------------
# Invariants that hold for any input (stated by the paper or implied by it).
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("seed,G,S,M,E,C,variant_a", [
    (0, 2, 64, 16, 8, 16, False), (1, 3, 100, 8, 5, 7, False), (2, 1, 257, 12, 16, 3, True),
    (3, 2, 128, 8, 2, 128, False), (4, 2, 96, 8, 32, 1, False)])
def test_invariants(seed, G, S, M, E, C, variant_a):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((G, S, M)).astype(np.float32)
    wg = (rng.standard_normal((M, E)) * 1.5).astype(np.float32)
    u = rng.random((G, S)).astype(np.float32)
    f = orc.forward(x, wg, None, None, u, C, variant_a=variant_a, want_y=False)
    for g in range(G):
        kept1 = f.slot[g, :, 0] >= 0
        kept2 = f.slot[g, :, 1] >= 0
        assert f.first_count[g].sum() == S
        if not variant_a:
            assert f.total_count[g].sum() == 2 * S
        else:
            assert f.total_count[g].sum() == S + ((f.flags[g] & 2) != 0).sum()
        assert f.m[g].sum() == pytest.approx(1.0, rel=1e-12)
        np.testing.assert_allclose(f.weight[g].sum(axis=1), 1.0, rtol=1e-12)
        assert np.all(f.weight[g, :, 0] >= 0.5)
        assert np.all(f.expert_idx[g, :, 0] != f.expert_idx[g, :, 1])
        for e in range(E):
            s1 = np.nonzero((f.expert_idx[g, :, 0] == e) & kept1)[0]
            s2 = np.nonzero((f.expert_idx[g, :, 1] == e) & kept2)[0]
            pos = np.concatenate([f.slot[g, s1, 0], f.slot[g, s2, 1]])
            assert len(pos) <= C                                  # at most C tokens per expert
            assert len(set(pos.tolist())) == len(pos)             # distinct buffer positions
            # kept first choices fill positions 0..min(c1,C)-1 in token order
            n1 = min(int(f.first_count[g, e]), C)
            assert f.slot[g, s1, 0].tolist() == list(range(n1))
            # an expert that is full after the first loop accepts no second choice
            if f.first_count[g, e] >= C:
                assert len(s2) == 0
            # slot_token is the exact inverse of slot
            inv = np.full(C, -1)
            inv[f.slot[g, s1, 0]] = s1
            inv[f.slot[g, s2, 1]] = s2
            assert f.slot_token[e, g].tolist() == inv.tolist()
        assert np.all((f.flags[g] & 4 == 0) | (f.flags[g] & 2 != 0))   # kept second => test passed
    assert f.l_aux == pytest.approx(f.l_aux_group.mean(), rel=1e-12)


# ---------------------------------------------------------------------------
# Closed forms.
# ---------------------------------------------------------------------------
def test_zero_gating_weights_closed_form():
    # wg = 0: all gates 1/E, every token picks (0,1) with w = 1/2,1/2 and passes the
    # random test; tokens 0..C-1 get y = (FFN_0 + FFN_1)/2, the rest 0; l_aux = 1/E^2.
    rng = np.random.default_rng(11)
    G, S, M, H, E, C = 2, 12, 6, 10, 4, 5
    x = rng.standard_normal((G, S, M)).astype(np.float32)
    wi = rng.standard_normal((E, M, H)).astype(np.float32)
    wo = rng.standard_normal((E, H, M)).astype(np.float32)
    u = rng.random((G, S)).astype(np.float32)
    f = orc.forward(x, np.zeros((M, E), np.float32), wi, wo, u, C)
    assert np.all(f.expert_idx[..., 0] == 0) and np.all(f.expert_idx[..., 1] == 1)
    assert f.l_aux == pytest.approx(1.0 / E ** 2, rel=1e-12)
    xd = x.astype(np.float64)
    ffn = [np.maximum(xd @ wi[e].astype(np.float64), 0) @ wo[e].astype(np.float64) for e in (0, 1)]
    expect = 0.5 * (ffn[0] + ffn[1])
    expect[:, C:, :] = 0.0
    np.testing.assert_allclose(f.y, expect, rtol=1e-10, atol=1e-12)


def test_two_experts_no_drop_is_dense_softmax_mixture():
    # E=2, C=S, u=0: nothing is dropped, w_k = p_k, so y = p0*FFN_0(x) + p1*FFN_1(x).
    rng = np.random.default_rng(12)
    G, S, M, H, E = 1, 20, 5, 9, 2
    x = rng.standard_normal((G, S, M)).astype(np.float32)
    wg = rng.standard_normal((M, E)).astype(np.float32)
    wi = rng.standard_normal((E, M, H)).astype(np.float32)
    wo = rng.standard_normal((E, H, M)).astype(np.float32)
    f = orc.forward(x, wg, wi, wo, np.zeros((G, S), np.float32), C=S)
    xd = x[0].astype(np.float64)
    logits = xd @ wg.astype(np.float64)
    p = np.exp(logits - logits.max(1, keepdims=True))
    p /= p.sum(1, keepdims=True)
    y = sum(p[:, [e]] * (np.maximum(xd @ wi[e].astype(np.float64), 0) @ wo[e].astype(np.float64))
            for e in range(E))
    np.testing.assert_allclose(f.y[0], y, rtol=1e-10, atol=1e-12)
    assert np.all(f.slot >= 0)


def test_l_aux_closed_forms():
    # identical tokens: every first choice goes to argmax p, so l_aux = p_max / E.
    S, E = 10, 4
    p = np.tile(np.array([[0.1, 0.2, 0.6, 0.1]]), (S, 1))
    e1, e2, g1, g2, _ = orc.top2(p)
    r = orc.capacity(E, 3, e1, e2, g1, g2, np.zeros(S, np.float32), orc.mean_gates(p))
    assert r.l_aux == pytest.approx(0.6 / E, rel=1e-12)
    # perfectly balanced first choices with uniform mean gates: l_aux = 1/E^2.
    S = 8
    p = np.full((S, E), 0.2)
    for s in range(S):
        p[s, s % E] = 0.4
    e1, e2, g1, g2, _ = orc.top2(p)
    r = orc.capacity(E, 4, e1, e2, g1, g2, np.zeros(S, np.float32), orc.mean_gates(p))
    assert r.first_count.tolist() == [2, 2, 2, 2]
    assert r.l_aux == pytest.approx(1.0 / E ** 2, rel=1e-12)


def test_softmax_gates_against_library():
    # the gating step reduces to a library matmul plus the textbook softmax.
    rng = np.random.default_rng(5)
    S, M, E = 33, 17, 11
    x = rng.standard_normal((S, M)).astype(np.float32)
    wg = rng.standard_normal((M, E)).astype(np.float32)
    logits, p = orc.gates(x, wg)
    ref = x.astype(np.float64) @ wg.astype(np.float64)
    np.testing.assert_allclose(logits, ref, rtol=1e-12, atol=1e-13)
    from scipy.special import softmax
    np.testing.assert_allclose(p, softmax(ref, axis=1), rtol=1e-12)
    np.testing.assert_allclose(orc.mean_gates(p), p.mean(axis=0), rtol=1e-13)
    # large logits must not overflow
    _, p_big = orc.gates(x * 1000.0, wg)
    assert np.all(np.isfinite(p_big)) and np.allclose(p_big.sum(1), 1.0)


def test_ffn_rows_against_library():
    rng = np.random.default_rng(6)
    R, M, H = 7, 12, 29                          # M != H catches a transposed operand
    xr = rng.standard_normal((R, M)).astype(np.float32)
    wi = rng.standard_normal((M, H)).astype(np.float32)
    wo = rng.standard_normal((H, M)).astype(np.float32)
    out, h = orc.ffn_rows(xr, wi, wo, want_h=True)
    href = xr.astype(np.float64) @ wi.astype(np.float64)
    np.testing.assert_allclose(h, href, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(out, np.maximum(href, 0) @ wo.astype(np.float64), rtol=1e-12, atol=1e-12)
