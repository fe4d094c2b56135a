"""Pins for the reporting pieces: reuse mass (Eq. 2), #uMiss/uHR aggregates (App. E.2.4), the I/O-time
and TPOT proxy (App. E.2.6, F.1), routing entropy and load-balance CV (Sec. 4.4, 5.2)."""
import os

import numpy as np

from oracle import remoe_oracle as orc
import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_cache_tables.txt")
TOTAL_REQUESTS = 128 * 64 * 26 * 6


def _balance_rows():
    rows = []
    for line in open(GOLDEN):
        c = [x.strip() for x in line.strip().split("|")]
        if c[0] == "balance":
            rows.append((int(c[1]), float(c[2]), float(c[3])))
    return rows


def _tables():
    cache, tpot = {}, {}
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        c = [x.strip() for x in line.split("|")]
        if c[0] == "balance":
            continue
        if c[0] == "tpot50":
            tpot[int(c[1])] = (float(c[2]), float(c[3]))
        else:
            cache[int(c[0])] = tuple(float(x) for x in c[1:])
    return cache, tpot


def test_uhr_and_umiss_definitions_reproduce_the_papers_table():
    """uHR = hits / (hits + misses) and #uMiss = misses, with hits + misses = layers*K*steps: feeding
    the oracle's counters with the paper's miss totals must give back the paper's hit rates."""
    cache, _ = _tables()
    shape = synth.Shape(26, 8, 64, 6, 8)
    for C, (uhr_b, um_b, uhr_r, um_r) in cache.items():
        for uhr, um in ((uhr_b, um_b), (uhr_r, um_r)):
            st = orc.OracleStack(shape, C, [np.zeros((64, 8))] * 26)
            misses = round(um * 1e6)
            st.uniq_misses[0] = misses
            st.uniq_hits[0] = TOTAL_REQUESTS - misses
            assert abs(st.uhr() - uhr) <= 1e-4 and abs(st.uhr(0) - uhr) <= 1e-4
            assert abs((1.0 - uhr) * TOTAL_REQUESTS / 1e6 - um) <= 2e-4


def test_tpot_proxy_scale_against_the_papers_table():
    """The proxy is linear in the misses with slope expert_bytes / bandwidth per miss.  Between cache
    sizes the paper's median TPOT moves by about that slope times the change in mean misses per step
    (medians against means: a few per cent of slack), for a DeepSeek-V2-Lite expert (3*2048*1408 bf16
    values) at 4.0 GB/s.  A wrong unit (s for ms, bits for bytes, a missing /B) is off by far more."""
    cache, tpot = _tables()
    expert_bytes = 3 * 2048 * 1408 * 2
    per_miss = float(orc.io_ms_step([1], expert_bytes, 4.0)[0])
    assert abs(per_miss - 4.325376) < 1e-9
    steps = 128 * 64
    for col in (0, 1):
        d_tpot = tpot[4][col] - tpot[12][col]
        d_miss = (cache[4][1 + 2 * col] - cache[12][1 + 2 * col]) * 1e6 / steps
        assert abs(d_tpot / d_miss / per_miss - 1.0) < 0.06
    t, pct = orc.tpot_proxy([10, 20, 30], expert_bytes, 4.0, batch=2, tpot_compute_ms=5.0)
    assert np.allclose(t, 5.0 + np.array([10, 20, 30]) * per_miss / 2)
    assert abs(pct[0] - t[1]) < 1e-12


def test_percentiles_match_numpy():
    rng = np.random.default_rng(0)
    um = rng.integers(0, 157, size=333)
    t, pct = orc.tpot_proxy(um, 1000, 1.0)
    assert np.allclose(pct, np.percentile(t, [50, 95, 99]), rtol=1e-12)
    _, one = orc.tpot_proxy([7], 1000, 1.0)
    assert one[0] == one[1] == one[2]


def test_reuse_mass_identities():
    p = orc.softmax(np.random.default_rng(1).standard_normal(16))
    assert abs(orc.reuse_mass(p, range(16), 4) - 1.0 / 4) < 1e-15           # all experts: sum P = 1
    assert abs(orc.reuse_mass(np.full(16, 1 / 16), [3, 5, 9, 11], 4) - 1 / 16) < 1e-15
    assert orc.reuse_mass(p, [], 4) == 0.0
    assert abs(orc.reuse_mass(p, [2, 7], 2) - (p[2] + p[7]) / 2) < 1e-15


def test_stack_tracks_mass_and_history():
    shape = synth.Shape(2, 64, 16, 3, 8, batch=2)
    routers = [synth.gen_router(0, shape, l) for l in range(2)]
    st = orc.OracleStack(shape, 6, routers)
    hs = synth.HiddenStream(0, shape, 0.6)
    prev = None
    for t in range(12):
        h = hs.step()
        r = st.step(h, ffn=None)
        if t == 0:
            assert (r["mass"] == -1).all()
        else:
            for l in range(2):
                for b in range(2):
                    p = orc.softmax(orc.router_logits(routers[l], h[l, b]))
                    assert abs(r["mass"][l, b] - sum(p[e] for e in prev[l, b]) / 3) < 1e-15
                    # the overlap counts the same experts with weight 1 instead of P
                    assert (r["overlap"][l, b] == 3) == (set(prev[l, b]) == set(r["ids"][l, b]))
        prev = r["ids"].copy()
    assert len(st.hist_umiss) == 12 and sum(st.hist_umiss) == sum(st.uniq_misses)
    assert sum(st.hist_tok_hits) == sum(st.tok_hits)


def test_load_entropy_and_cv_closed_forms():
    n = 64
    assert abs(orc.load_entropy([7] * n) - 1.0) < 1e-12 and orc.load_cv([7] * n) == 0.0
    one_hot = [0] * n
    one_hot[5] = 123
    assert abs(orc.load_entropy(one_hot)) < 1e-15
    assert abs(orc.load_cv(one_hot) - np.sqrt(n - 1)) < 1e-12
    # m of N experts share the load evenly: entropy log m / log N, CV sqrt(N / m - 1)
    for m in (2, 16, 48):
        c = [3] * m + [0] * (n - m)
        assert abs(orc.load_entropy(c) - np.log(m) / np.log(n)) < 1e-12
        assert abs(orc.load_cv(c) - np.sqrt(n / m - 1)) < 1e-12
    # half the experts at mean * (1 + c), half at mean * (1 - c): CV = c exactly and
    # H = log N - ((1 + c) log(1 + c) + (1 - c) log(1 - c)) / 2
    for c in (0.0409, 0.1608, 0.5):
        counts = [round(1e6 * (1 + c))] * 32 + [round(1e6 * (1 - c))] * 32
        assert abs(orc.load_cv(counts) - c) < 1e-9
        h = 1.0 - ((1 + c) * np.log(1 + c) + (1 - c) * np.log(1 - c)) / (2 * np.log(64))
        assert abs(orc.load_entropy(counts) - h) < 1e-9
    # invariances: scale of the counts, order of the experts
    rng = np.random.default_rng(3)
    v = rng.integers(1, 1000, size=60)
    assert abs(orc.load_entropy(v) - orc.load_entropy(3 * v)) < 1e-12
    assert abs(orc.load_cv(v) - orc.load_cv(rng.permutation(v) * 5)) < 1e-12
    assert abs(orc.load_cv(v) - np.std(v) / np.mean(v)) < 1e-12
    assert orc.load_entropy([0] * 8) == 1.0 and orc.load_cv([0] * 8) == 0.0        # nothing routed yet


def test_entropy_and_cv_readings_fit_the_pairs_the_paper_prints():
    """The paper prints entropy and CV without formulas.  With entropy read as H(load) / log N and CV
    as std / mean of the per-expert load, the two are tied near balance by
    H / log N = 1 - CV^2 / (2 log N) + O(CV^3); every printed pair obeys that to its last digit or
    two, for both expert counts.  (A per-token softmax entropy, an unnormalised entropy or a CV of
    something other than the load would not.)"""
    rows = _balance_rows()
    assert len(rows) == 8
    for n, ent, cv in rows:
        assert abs(ent - (1.0 - cv * cv / (2.0 * np.log(n)))) < (6e-5 if cv < 0.06 else 4e-4)
    # and the oracle's own functions obey the same relation on a mildly perturbed load
    rng = np.random.default_rng(7)
    counts = np.round(1e5 * (1 + 0.1 * rng.standard_normal(64))).astype(np.int64)
    cv = orc.load_cv(counts)
    assert abs(orc.load_entropy(counts) - (1.0 - cv * cv / (2 * np.log(64)))) < 2e-4


def test_stack_counts_the_load_per_expert():
    shape = synth.Shape(2, 64, 16, 3, 8, batch=2)
    routers = [synth.gen_router(0, shape, l) for l in range(2)]
    st = orc.OracleStack(shape, 6, routers)
    hs = synth.HiddenStream(0, shape, 0.6)
    tally = np.zeros((2, 16), np.int64)
    for t in range(20):
        r = st.step(hs.step(), ffn=None)
        for l in range(2):
            for e in r["ids"][l].reshape(-1):
                tally[l, e] += 1
    assert (np.asarray(st.load) == tally).all() and tally.sum() == 20 * 2 * 2 * 3
    assert abs(st.routing_entropy() - (orc.load_entropy(tally[0]) + orc.load_entropy(tally[1])) / 2) < 1e-15
    assert abs(st.routing_cv(1) - np.std(tally[1]) / np.mean(tally[1])) < 1e-12
    assert st.experts_visited(0) == (tally[0] > 0).sum()
    st.reset()
    assert np.asarray(st.load).sum() == 0
