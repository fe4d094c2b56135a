"""Pins for the oracle's routing pieces (Sec. 3.1): logits, softmax, top-K, gate weights."""
import itertools
import math

import numpy as np
import pytest

from oracle import remoe_oracle as orc


def test_logits_match_explicit_loops():
    rng = np.random.default_rng(0)
    w = rng.standard_normal((5, 7))
    h = rng.standard_normal(7)
    z = orc.router_logits(w, h)
    for i in range(5):
        acc = 0.0
        for j in range(7):
            acc += w[i, j] * h[j]
        assert abs(z[i] - acc) < 1e-12
    # one row per expert: a one-hot h picks out a column of W_r
    e3 = np.zeros(7); e3[3] = 1.0
    assert np.array_equal(orc.router_logits(w, e3), w[:, 3])


def test_softmax_closed_forms():
    assert np.array_equal(orc.softmax(np.full(16, 3.25)), np.full(16, 1.0 / 16))
    a, b = 0.3, -1.1
    p = orc.softmax([a, b])
    assert abs(p[0] - 1.0 / (1.0 + math.exp(b - a))) < 1e-15
    z = np.random.default_rng(1).standard_normal(60) * 5
    p = orc.softmax(z)
    assert abs(p.sum() - 1.0) <= 1e-6
    assert np.allclose(orc.softmax(z + 1234.5), p, rtol=1e-12, atol=0)
    assert np.all(np.diff(p[np.argsort(z)]) >= 0)            # monotone in z
    # ratio identity P_i / P_j = exp(z_i - z_j)
    assert abs(p[4] / p[9] - math.exp(z[4] - z[9])) < 1e-12 * p[4] / p[9] + 1e-15
    # large logits do not overflow
    assert np.isfinite(orc.softmax([1000.0, 999.0])).all()


def test_softmax_matches_library():
    sp = pytest.importorskip("scipy.special")
    z = np.random.default_rng(2).standard_normal(128) * 3
    assert np.allclose(orc.softmax(z), sp.softmax(z), rtol=1e-13, atol=0)


def _topk_by_definition(z, k):
    """e is selected iff fewer than k experts beat it, where j beats e when
    z_j > z_e, or z_j == z_e and j < e."""
    n = len(z)
    sel = []
    for e in range(n):
        beats = sum(1 for j in range(n) if z[j] > z[e] or (z[j] == z[e] and j < e))
        if beats < k:
            sel.append((beats, e))
    return [e for _, e in sorted(sel)]


@pytest.mark.parametrize("n,k", [(1, 1), (5, 2), (16, 2), (33, 6), (60, 4), (64, 6), (128, 8), (7, 7)])
def test_topk_against_definition(n, k):
    rng = np.random.default_rng(n * 100 + k)
    for trial in range(20):
        z = rng.standard_normal(n)
        if trial % 2:
            z = np.round(z * 2) / 2                 # many exact ties
        ids, margin = orc.topk_select(z, k)
        assert list(ids) == _topk_by_definition(z, k)
        if k < n:
            rest = np.delete(z, ids)
            assert margin == z[ids[-1]] - rest.max()
            assert margin >= 0
        else:
            assert margin == float("inf")


def test_topk_constructed_ties():
    z = np.array([1.0, 2.0, 2.0, 0.5, 2.0, 1.0])
    ids, margin = orc.topk_select(z, 2)
    assert list(ids) == [1, 2] and margin == 0.0
    ids, _ = orc.topk_select(z, 4)
    assert list(ids) == [1, 2, 4, 0]
    ids, _ = orc.topk_select(np.zeros(9), 3)
    assert list(ids) == [0, 1, 2]


def test_topk_all_permutations_small():
    for perm in itertools.permutations([0.1, 0.2, 0.2, 0.4]):
        z = np.array(perm)
        for k in (1, 2, 3):
            assert list(orc.topk_select(z, k)[0]) == _topk_by_definition(z, k)


def test_gate_weights():
    z = np.random.default_rng(3).standard_normal(64)
    p = orc.softmax(z)
    ids, _ = orc.topk_select(z, 6)
    g = orc.gate_weights(p, ids, renorm=False)
    assert np.array_equal(g, p[ids]) and g.sum() <= 1.0
    assert np.all(np.diff(g) <= 0)                 # ordered by descending probability
    gr = orc.gate_weights(p, ids, renorm=True)
    assert abs(gr.sum() - 1.0) < 1e-12
    assert np.allclose(gr / gr[0], g / g[0], rtol=1e-13)
    ids_all, _ = orc.topk_select(z, 64)
    assert abs(orc.gate_weights(p, ids_all, False).sum() - 1.0) <= 1e-6


def test_unique_in_order_and_overlap():
    assert orc.unique_in_order([5, 3, 5, 1, 3, 9]) == [5, 3, 1, 9]
    assert orc.unique_in_order([]) == []
    assert orc.reuse_overlap([1, 2, 3], [3, 4, 1]) == 2
    assert orc.reuse_overlap([1, 2], [3, 4]) == 0
    assert orc.reuse_overlap([7, 8], [8, 7]) == 2


def test_near_tie_rule_of_the_parity_harness():
    """What the GPU parity tests accept as a near-tie: lists that differ only where two oracle logits
    are closer than 1e-5 (boundary flip or two ranks swapped), nothing else."""
    from parity_util import near_tie_kind, near_tie_only
    z = np.array([3.0, 2.0, 2.0 - 4e-6, 1.0, 1.0 - 2e-6, -5.0])
    ids, _ = orc.topk_select(z, 4)
    assert list(ids) == [0, 1, 2, 3]
    assert near_tie_only(z, ids, [0, 2, 1, 3])            # ranks 2 and 3 swapped across a 4e-6 gap
    assert near_tie_only(z, ids, [0, 1, 2, 4])            # boundary: expert 4 instead of 3, 2e-6 apart
    assert near_tie_only(z, ids, [0, 2, 1, 4])
    assert not near_tie_only(z, ids, [1, 0, 2, 3])        # a gap of 1.0 is not a tie
    assert not near_tie_only(z, ids, [0, 1, 2, 5])
    assert not near_tie_only(z, ids, [0, 1, 3, 2])        # 2 and 3 are 1.0 apart
    # a valid list holds K distinct ids inside [0, N): near-tied logits excuse none of these
    assert not near_tie_only(z, ids, [0, 1, 1, 3])        # expert 1 twice (1 and 2 are near-tied)
    assert not near_tie_only(z, ids, [0, 2, 2, 3])
    assert not near_tie_only(z, ids, [0, 1, 2, 6]) and not near_tie_only(z, ids, [0, 1, 2, -1])
    assert not near_tie_only(z, ids, [0, 1, 2]) and not near_tie_only(z, ids, [0, 1, 2, 3, 4])
    # and the two accepted kinds are told apart
    assert near_tie_kind(z, ids, [0, 1, 2, 3]) == "same"
    assert near_tie_kind(z, ids, [0, 2, 1, 3]) == "swap"
    assert near_tie_kind(z, ids, [0, 1, 2, 4]) == "boundary"
    assert near_tie_kind(z, ids, [0, 2, 1, 4]) == "boundary"
    assert near_tie_kind(z, ids, [1, 0, 2, 3]) is None
