"""Pins for three pieces of the stepped oracle that the other files reach only through the GPU:
the cache-aware rerouting branch of `OracleStack.route` (App. F.2), the token hit rate `thr`
(App. E.2.4) and the line of `OracleStack.step` that forms the shared expert's sigmoid gate from
the layer input.  Each is set against something worked out here by hand or fixed by the paper's
definitions, so that a wrong sign, a bonus applied to the wrong experts, a gate taken from the
biased scores, a hit rate over the wrong denominator or a gate formed from the wrong vector fails.
"""
import math
from types import SimpleNamespace

import numpy as np

from oracle import remoe_oracle as orc


def _shape(**kw):
    base = dict(n_layers=1, hidden=8, n_routed=6, top_k=2, inter_routed=4, n_shared=0, inter_shared=0,
                shared_gate=0, renorm_topk=0, weight_dtype=0, batch=1)
    base.update(kw)
    return SimpleNamespace(**base)


def _unit_router(n, h):
    """Router whose logit of expert e is simply x[e]."""
    w = np.zeros((n, h))
    for e in range(n):
        w[e, e] = 1.0
    return w


# ------------------------------------------------------------------ rerouting bonus (App. F.2)

def test_reroute_zero_bonus_is_the_plain_router():
    rng = np.random.default_rng(3)
    s = _shape(n_routed=12, hidden=16, top_k=3)
    wr = rng.standard_normal((12, 16))
    a = orc.OracleStack(s, 4, [wr])
    b = orc.OracleStack(s, 4, [wr], reroute_beta=0.0)
    c = orc.OracleStack(s, 4, [wr], reroute_beta=1e-300)        # non-zero but far below any logit gap
    for t in range(40):
        h = rng.standard_normal((1, 1, 16))
        ra, rb, rc = a.step(h, ffn=None), b.step(h, ffn=None), c.step(h, ffn=None)
        assert np.array_equal(ra["ids"], rb["ids"]) and np.array_equal(ra["ids"], rc["ids"])
        assert np.array_equal(ra["gates"], rb["gates"]) and np.array_equal(ra["gates"], rc["gates"])
        assert ra["hit"] == rb["hit"] == rc["hit"] and ra["slot"] == rb["slot"] == rc["slot"]


def test_reroute_hand_worked_steps():
    """Logits are the inputs themselves (unit router), N = 6, K = 2, C = 3, beta = 1.
    Step 1, x = (5, 4, 3, 2, 1, 0), cold cache: no bonus anywhere -> E = [0, 1], both misses.
    Step 2, x = (0, 3.5, 4.2, 4, 1, 0), residents {0, 1}: scores (1, 4.5, 4.2, 4, 1, 0) -> E = [1, 2]
      (plain routing would give [2, 3]); gates are the UNBIASED softmax at 1 and 2.
    Step 3, x = (0, 0, 0, 0.9, 0.5, 0), residents {0, 1, 2}: scores (1, 1, 1, 0.9, 0.5, 0) -> the tie
      between 0, 1, 2 goes to the lower indices: E = [0, 1]; plain routing would give [3, 4].
    """
    s = _shape()
    st = orc.OracleStack(s, 3, [_unit_router(6, 8)], reroute_beta=1.0)
    x1 = np.array([5, 4, 3, 2, 1, 0, 0, 0], float)
    x2 = np.array([0, 3.5, 4.2, 4, 1, 0, 0, 0], float)
    x3 = np.array([0, 0, 0, 0.9, 0.5, 0, 0, 0], float)
    r1 = st.step(x1.reshape(1, 1, 8), ffn=None)
    assert list(r1["ids"][0, 0]) == [0, 1] and r1["hit"][0] == [False, False]
    r2 = st.step(x2.reshape(1, 1, 8), ffn=None)
    assert list(r2["ids"][0, 0]) == [1, 2]
    assert r2["hit"][0] == [True, False] and r2["slot"][0] == [1, 2]
    p2 = np.exp(x2[:6]) / np.exp(x2[:6]).sum()                   # softmax of the unbiased logits
    assert np.allclose(r2["gates"][0, 0], [p2[1], p2[2]], rtol=1e-14)
    assert not np.isclose(r2["gates"][0, 0][0], math.exp(4.5) / (np.exp([1, 4.5, 4.2, 4, 1, 0]).sum()))
    r3 = st.step(x3.reshape(1, 1, 8), ffn=None)
    assert list(r3["ids"][0, 0]) == [0, 1] and r3["hit"][0] == [True, True]
    # the same three inputs without the bonus
    plain = orc.OracleStack(s, 3, [_unit_router(6, 8)])
    got = [list(plain.step(x.reshape(1, 1, 8), ffn=None)["ids"][0, 0]) for x in (x1, x2, x3)]
    assert got == [[0, 1], [2, 3], [3, 4]]


def test_reroute_large_bonus_freezes_the_selection():
    """A bonus above the whole logit range puts every resident expert ahead of every other one.  With
    C = K the cache holds exactly the first step's experts, so every later step selects that same set
    (in the order of its current logits), never misses, IR = 1, and the gate weights are still the
    plain softmax probabilities of those experts."""
    rng = np.random.default_rng(5)
    N, H, K = 10, 12, 3
    s = _shape(n_routed=N, hidden=H, top_k=K)
    wr = rng.standard_normal((N, H))
    st = orc.OracleStack(s, K, [wr], reroute_beta=1e3)
    first = None
    for t in range(30):
        h = rng.standard_normal(H)
        r = st.step(h.reshape(1, 1, H), ffn=None)
        ids = [int(e) for e in r["ids"][0, 0]]
        z = wr @ h
        p = np.exp(z - z.max()) / np.exp(z - z.max()).sum()
        if t == 0:
            first = set(ids)
            assert ids == sorted(range(N), key=lambda i: (-z[i], i))[:K]      # cold cache: plain top-K
            assert r["hit"][0] == [False] * K
        else:
            assert set(ids) == first
            assert ids == sorted(first, key=lambda i: (-z[i], i))
            assert r["hit"][0] == [True] * K and r["overlap"][0, 0] == K
        assert np.allclose(r["gates"][0, 0], [p[i] for i in ids], rtol=1e-13)
    assert st.uniq_misses[0] == K and st.eor() == 1.0


def test_reroute_bonus_goes_to_residents_of_the_state_before_the_step():
    """C = 4 > K = 2: an expert admitted two steps ago and not used since still gets the bonus, an
    expert evicted meanwhile does not.  Unit router, beta = 2."""
    s = _shape()
    st = orc.OracleStack(s, 4, [_unit_router(6, 8)], reroute_beta=2.0)

    def go(x6):
        x = np.zeros(8)
        x[:6] = x6
        return st.step(x.reshape(1, 1, 8), ffn=None)

    go([9, 8, 0, 0, 0, 0])                       # admits 0, 1
    go([0, 0, 9, 8, 0, 0])                       # residents 0, 1 get +2 -> (2, 2, 9, 8): admits 2, 3
    r = go([1, 0, 0, 0, 2.5, 2.4])               # residents {0,1,2,3}: scores (3, 2, 2, 2, 2.5, 2.4)
    assert list(r["ids"][0, 0]) == [0, 4]        # resident 0 wins through the bonus; 4 beats 5 and the 2s
    assert r["hit"][0] == [True, False] and r["evicted"][0][1] == 1     # LRU victim: expert 1
    r = go([0, 2.2, 0, 0, 0, 0.1])               # 1 is no longer resident: scores (2, 2.2, 2, 2, 2, 0.1)
    assert list(r["ids"][0, 0]) == [1, 0]
    assert r["hit"][0] == [False, True]


# ------------------------------------------------------------------ token hit rate (App. E.2.4)

def test_thr_and_uhr_on_a_hand_counted_batched_run():
    """B = 3 sequences, K = 2, N = 6, C = 3, unit router so the selections can be read off the inputs.
    Step 1 selects (0,1) (0,2) (0,1): R = [0,1,0,2,0,1], cache empty -> 0 of 6 token hits, U = [0,1,2],
      3 unique misses; cache becomes {0,1,2}.
    Step 2 selects (0,1) (3,0) (4,5): R = [0,1,3,0,4,5] -> token hits 0,1,0 = 3 of 6; U = [0,1,3,4,5]:
      2 unique hits, 3 unique misses.
    tHR = 3/12, uHR = 2/8."""
    s = _shape(batch=3)
    st = orc.OracleStack(s, 3, [_unit_router(6, 8)])

    def rows(sel):
        h = np.zeros((1, 3, 8))
        for b, (first, second) in enumerate(sel):
            h[0, b, first], h[0, b, second] = 2.0, 1.0
        return h

    r1 = st.step(rows([(0, 1), (0, 2), (0, 1)]), ffn=None)
    assert r1["requests"][0] == [0, 1, 2] and r1["tok_hits"] == [0]
    r2 = st.step(rows([(0, 1), (3, 0), (4, 5)]), ffn=None)
    assert r2["requests"][0] == [0, 1, 3, 4, 5] and r2["tok_hits"] == [3]
    assert r2["hit"][0] == [True, True, False, False, False]
    assert (st.tok_hits[0], st.tok_misses[0]) == (3, 9)
    assert (st.uniq_hits[0], st.uniq_misses[0]) == (2, 6)
    assert st.thr() == 3 / 12 and st.thr(0) == 3 / 12
    assert st.uhr() == 2 / 8 and st.uhr(0) == 2 / 8
    assert orc.OracleStack(s, 3, [_unit_router(6, 8)]).thr() == 0.0          # nothing served yet


def test_thr_sums_counts_over_layers_not_rates():
    """Two layers with different traffic: the all-layer rate is the ratio of summed counts
    (App. E.2.4 "summing counts across MoE layers"), not the mean of the per-layer rates."""
    s = _shape(n_layers=2, batch=2)
    st = orc.OracleStack(s, 4, [_unit_router(6, 8), _unit_router(6, 8)])
    h = np.zeros((2, 2, 8))
    h[0, 0, [0, 1]] = [2, 1]; h[0, 1, [0, 1]] = [2, 1]          # layer 0: both sequences pick (0, 1)
    h[1, 0, [2, 3]] = [2, 1]; h[1, 1, [4, 5]] = [2, 1]          # layer 1: (2, 3) and (4, 5)
    st.step(h, ffn=None)
    h2 = h.copy()
    h2[1] = 0.0
    h2[1, 0, [2, 0]] = [2, 1]; h2[1, 1, [1, 0]] = [2, 1]        # layer 1 now (2, 0) and (1, 0)
    st.step(h2, ffn=None)
    # layer 0: step 2 all four token requests hit -> 4 / 8; layer 1: only expert 2 hits -> 1 / 8
    assert st.thr(0) == 4 / 8 and st.thr(1) == 1 / 8 and st.thr() == 5 / 16
    # unique level: layer 0 U = [0,1] twice -> 2 hits of 4; layer 1 U = [2,3,4,5] then [2,0,1] -> 1 of 7
    assert st.uhr(0) == 2 / 4 and st.uhr(1) == 1 / 7 and st.uhr() == 3 / 11
    assert st.uhr() != (st.uhr(0) + st.uhr(1)) / 2


# ------------------------------------------------------------------ shared-expert sigmoid gate

def _one_expert_weights(H, I, rng):
    return (rng.standard_normal((I, H)), rng.standard_normal((I, H)), rng.standard_normal((H, I)))


def test_shared_gate_scale_is_sigmoid_of_gate_vector_dot_layer_input():
    """One routed expert with zero weights and one shared expert: the layer output is
    sigmoid(w_sg . x) * y_shared(x).  With w_sg the j-th unit vector the scale must be sigmoid(x_j) --
    of this layer's input, of this sequence."""
    rng = np.random.default_rng(7)
    H, I = 8, 5
    s = _shape(n_layers=2, n_routed=1, top_k=1, n_shared=1, inter_shared=I, shared_gate=1, batch=2)
    zero = (np.zeros((4, H)), np.zeros((4, H)), np.zeros((H, 4)))
    shared = [_one_expert_weights(H, I, rng) for _ in range(2)]
    sg = [np.eye(H)[2], -3.0 * np.eye(H)[5]]                 # layer 0 reads x_2, layer 1 reads -3 x_5
    st = orc.OracleStack(s, 1, [np.ones((1, H)), np.ones((1, H))], lambda l, e: zero, lambda l, i: shared[l],
                         shared_gates=sg)
    h = rng.standard_normal((2, 2, H))
    r = st.step(h, ffn="dense")
    for l, (j, c) in enumerate([(2, 1.0), (5, -3.0)]):
        for b in range(2):
            want = 1.0 / (1.0 + math.exp(-c * h[l, b, j]))
            assert abs(r["shared_scale"][l, b] - want) < 1e-15
            y = orc.swiglu_expert(*shared[l], h[l, b])
            assert np.allclose(r["out"][l, b], want * y, rtol=1e-13, atol=1e-15)
    # without the flag the shared expert enters with weight 1 whatever the gate vectors hold
    s0 = _shape(n_layers=2, n_routed=1, top_k=1, n_shared=1, inter_shared=I, shared_gate=0, batch=2)
    r0 = orc.OracleStack(s0, 1, [np.ones((1, H))] * 2, lambda l, e: zero, lambda l, i: shared[l],
                         shared_gates=sg).step(h, ffn="dense")
    assert np.all(r0["shared_scale"] == 1.0)
    assert np.allclose(r0["out"][1, 0], orc.swiglu_expert(*shared[1], h[1, 0]), rtol=1e-13)


def test_shared_gate_scale_in_chained_mode_reads_the_normalised_input():
    """Chained mode feeds every layer x_l = h_l / sqrt(mean(h_l^2) + 1e-6); the gate must see x_l, not
    the residual stream h_l: with a unit gate vector the scale is sigmoid(x_l[j])."""
    rng = np.random.default_rng(9)
    H, I = 8, 5
    s = _shape(n_layers=2, n_routed=1, top_k=1, n_shared=1, inter_shared=I, shared_gate=1)
    zero = (np.zeros((4, H)), np.zeros((4, H)), np.zeros((H, 4)))
    shared = [_one_expert_weights(H, I, rng) for _ in range(2)]
    sg = [np.eye(H)[1], np.eye(H)[6]]
    st = orc.OracleStack(s, 1, [np.ones((1, H))] * 2, lambda l, e: zero, lambda l, i: shared[l], shared_gates=sg)
    h0 = 3.0 * rng.standard_normal((1, H))                    # far from unit RMS, so x != h
    r = st.step(h0, ffn="selected", chained=True)
    hl = h0[0].copy()
    for l, j in enumerate([1, 6]):
        x = hl / math.sqrt(float(np.mean(hl * hl)) + 1e-6)
        want = 1.0 / (1.0 + math.exp(-x[j]))
        assert abs(r["shared_scale"][l, 0] - want) < 1e-15
        assert abs(want - 1.0 / (1.0 + math.exp(-hl[j]))) > 1e-3          # the unnormalised reading differs
        hl = hl + want * orc.swiglu_expert(*shared[l], x)
    assert np.allclose(r["final"][0], hl, rtol=1e-13)
