"""Pins for the oracle's cache model (App. A.1-A.5, App. E.2) and reuse statistic (Eq. 1)."""
import itertools
import os

import numpy as np
import pytest

from oracle import remoe_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                yield [c.strip() for c in line.split("|")]


def test_lru_hand_trace():
    cache = orc.SlotCache(3)
    for req, hit, slot, ev in _rows("lru_hand_trace.txt"):
        req = [int(x) for x in req.split()]
        h, s, e = cache.serve(req)
        assert [int(x) for x in h] == [int(x) for x in hit.split()]
        assert s == [int(x) for x in slot.split()]
        assert e == [int(x) for x in ev.split()]


def test_fifo_lfu_hand_trace():
    caches = {"fifo": orc.SlotCache(2, "fifo"), "lfu": orc.SlotCache(2, "lfu")}
    for pol, req, hit, slot, ev in _rows("fifo_lfu_hand_trace.txt"):
        h, s, e = caches[pol].serve([int(req)])
        assert (int(h[0]), s[0], e[0]) == (int(hit), int(slot), int(ev))


def _random_trace(rng, n, k, steps, sticky):
    prev = list(rng.choice(n, k, replace=False))
    out = [prev]
    for _ in range(steps - 1):
        cur = [e for e in prev if rng.random() < sticky]
        pool = [e for e in range(n) if e not in cur]
        rng.shuffle(pool)
        cur = cur + pool[: k - len(cur)]
        rng.shuffle(cur)
        out.append([int(e) for e in cur])
        prev = cur
    return out


def _mru_set_from_history(log, capacity):
    """The `capacity` most recently used distinct experts of a full access log."""
    seen = []
    for e in reversed(log):
        if e not in seen:
            seen.append(e)
            if len(seen) == capacity:
                break
    return set(seen)


@pytest.mark.parametrize("n,k,c", [(8, 2, 2), (8, 2, 3), (16, 2, 4), (12, 3, 7), (64, 6, 16), (10, 4, 10)])
def test_lru_is_most_recently_used_set(n, k, c):
    """App. A.5: LRU preserves the most recently used distinct experts.  The resident set
    is recomputed from the whole access history at every step, independently of the
    incremental slot bookkeeping."""
    rng = np.random.default_rng(n * 1000 + k * 10 + c)
    cache = orc.SlotCache(c)
    log = []
    for req in _random_trace(rng, n, k, 200, sticky=0.5):
        before = _mru_set_from_history(log, c)
        assert cache.resident() == before
        hit, slot, evicted = cache.serve(req)
        assert hit == [e in before for e in req]                 # judged against C_t
        log += [e for e, h in zip(req, hit) if h] + [e for e, h in zip(req, hit) if not h]
        assert set(req) <= cache.resident()                      # E_t subset of C_{t+1}
        assert len(cache.resident()) <= c
        for e, s in zip(req, slot):
            assert cache.expert_of_slot[s] == e


def test_slot_rules():
    cache = orc.SlotCache(5)
    hit, slot, ev = cache.serve([9, 4, 7])                        # cold: lowest empty slots
    assert hit == [False] * 3 and slot == [0, 1, 2] and ev == [-1] * 3
    hit, slot, ev = cache.serve([7, 1, 9])
    assert hit == [True, False, True] and slot == [2, 3, 0] and ev == [-1, -1, -1]
    hit, slot, ev = cache.serve([2, 3])                           # one empty slot, then evict 4
    assert slot == [4, 1] and ev == [-1, 4]
    # a hit never moves; an evicted expert's slot is the one reused
    hit, slot, ev = cache.serve([9])
    assert hit == [True] and slot == [0]


@pytest.mark.parametrize("n,k", [(8, 2), (16, 4), (64, 6)])
def test_exact_miss_count_when_capacity_equals_k(n, k):
    """Tightness case of Prop. 3.1 / A.4: C = K gives misses(t) = K - |E_t n E_{t-1}|."""
    rng = np.random.default_rng(7 + n + k)
    trace = _random_trace(rng, n, k, 300, sticky=0.6)
    cache = orc.SlotCache(k)
    for t, req in enumerate(trace):
        hit, _, _ = cache.serve(req)
        misses = len(req) - sum(hit)
        if t == 0:
            assert misses == k                                    # cold start
        else:
            assert misses == k - orc.reuse_overlap(req, trace[t - 1])


@pytest.mark.parametrize("policy", ["lru", "fifo", "lfu"])
@pytest.mark.parametrize("n,k,c", [(16, 2, 4), (64, 6, 16), (60, 4, 12), (32, 8, 8)])
def test_fetch_bounds(policy, n, k, c):
    """Prop. 3.1: misses(t) <= K - |E_t n E_{t-1}| for C >= K (any admitting policy);
    longer-horizon bound misses(t) <= K - |E_t n U_{t,L_t}| for LRU (App. A.5)."""
    rng = np.random.default_rng(11 + n + k + c)
    trace = _random_trace(rng, n, k, 300, sticky=0.4)
    cache = orc.SlotCache(c, policy)
    for t, req in enumerate(trace):
        hit, _, _ = cache.serve(req)
        misses = len(req) - sum(hit)
        if t >= 1:
            assert misses <= k - orc.reuse_overlap(req, trace[t - 1])
            if policy == "lru":
                u, ell = set(), 0
                while t - ell - 1 >= 0 and len(u | set(trace[t - ell - 1])) <= c:
                    u |= set(trace[t - ell - 1])
                    ell += 1
                assert ell >= 1
                assert misses <= k - len(set(req) & u)
        assert set(req) <= cache.resident()


def test_full_capacity_misses_equal_distinct_experts():
    rng = np.random.default_rng(5)
    trace = _random_trace(rng, 16, 3, 100, sticky=0.2)
    cache = orc.SlotCache(16)
    misses = sum(len(r) - sum(cache.serve(r)[0]) for r in trace)
    assert misses == len(set(e for r in trace for e in r))


def test_more_requests_than_slots():
    """Same two-phase rule when |U| > C: the state ends as the last C entries of
    [hits..., misses...]; counts are still judged against the pre-step state."""
    cache = orc.SlotCache(3)
    cache.serve([1, 2, 3])
    hit, slot, ev = cache.serve([4, 2, 5, 6, 7])
    assert hit == [False, True, False, False, False]
    # hits first: 2 touched; then 4 evicts 1 (slot 0), 5 evicts 3 (slot 2), 6 evicts 2 (slot 1),
    # 7 evicts 4 (slot 0)
    assert slot == [0, 1, 2, 1, 0]
    assert ev == [1, -1, 3, 2, 4]
    assert cache.resident() == {5, 6, 7}


def _belady_exhaustive(steps, capacity):
    """Minimum misses over every eviction choice (tiny inputs only)."""
    best = [10 ** 9]

    def rec(t, resident, misses):
        if misses >= best[0]:
            return
        if t == len(steps):
            best[0] = misses
            return
        req = set(steps[t])
        misses += len(req - resident)
        pool = resident | req
        over = len(pool) - capacity
        if over <= 0:
            rec(t + 1, frozenset(pool), misses)
            return
        for drop in itertools.combinations(sorted(pool - req), over):
            rec(t + 1, frozenset(pool - set(drop)), misses)

    rec(0, frozenset(), 0)
    return best[0]


def test_belady_against_exhaustive_search():
    rng = np.random.default_rng(3)
    for _ in range(15):
        trace = _random_trace(rng, 6, 2, 9, sticky=0.3)
        for c in (2, 3, 4):
            assert orc.belady_min_misses(trace, c) == _belady_exhaustive(trace, c)
            lru = orc.SlotCache(c)
            lru_misses = sum(len(r) - sum(lru.serve(r)[0]) for r in trace)
            assert orc.belady_min_misses(trace, c) <= lru_misses
