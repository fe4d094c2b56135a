"""Helpers that set the CUDA library beside the CPU oracle on the same seeded inputs."""
from __future__ import annotations

import numpy as np

import synth
from oracle import remoe_oracle as orc

TOL = {0: 1e-4, 1: 2e-2, 2: 2e-2, 3: 2e-2}  # max|d| / max|ref| : float32, bf16, fp8, int4 weights (fp32 accumulate)
NEAR_TIE = 1e-5                   # logit gap below which the selected list may differ


def near_tie_kind(z, o_ids, ids):
    """How the library's list `ids` relates to the oracle's `o_ids` for the oracle logits `z`:
    "same", "boundary", "swap" or None (not acceptable).

    A list is acceptable only if it holds K distinct expert ids inside [0, N) and, at every rank, an
    expert whose oracle logit is within NEAR_TIE of the oracle's expert at that rank.  "boundary": the
    selected SET differs (rank K against rank K+1 -- the case the acceptance rule names); "swap": the
    same set with two near-tied ranks exchanged.  Both can only happen when fp32 rounding of the logits
    meets a gap that small (Top-K stability, App. C)."""
    o_ids = [int(e) for e in o_ids]
    ids = [int(e) for e in ids]
    n = len(z)
    if len(ids) != len(o_ids) or len(set(ids)) != len(ids) or any(e < 0 or e >= n for e in ids):
        return None
    if ids == o_ids:
        return "same"
    if not all(abs(float(z[a]) - float(z[b])) < NEAR_TIE for a, b in zip(o_ids, ids)):
        return None
    return "swap" if set(ids) == set(o_ids) else "boundary"


def near_tie_only(z, o_ids, ids):
    """True if `ids` is the oracle's list or differs from it only by near-ties (see near_tie_kind)."""
    return near_tie_kind(z, o_ids, ids) is not None


def widen(shape, a, router=False):
    return synth.widen(shape, a, router)


def oracle_for(wl, policy="lru", reroute_beta=0.0):
    """An OracleStack reading the very arrays the library was loaded from."""
    s = wl.shape
    routers = [widen(s, r, True) for r in wl.routers]
    sg = None if wl.shared_gates is None else [widen(s, g, True) for g in wl.shared_gates]

    def ew(l, e):
        return synth.expert_matrices(widen(s, wl.expert_block(l, e)), s.hidden, s.inter_routed)

    def sw(l, i):
        return synth.expert_matrices(widen(s, wl.shared[l][i]), s.hidden, s.inter_shared)

    return orc.OracleStack(s, wl.cache_slots, routers, ew, sw, shared_gates=sg, policy=policy,
                           reroute_beta=reroute_beta)


def rel_err(got, ref):
    ref = np.asarray(ref, dtype=np.float64)
    denom = np.max(np.abs(ref))
    return float(np.max(np.abs(np.asarray(got, dtype=np.float64) - ref)) / (denom if denom > 0 else 1.0))


class StepChecker:
    """Feeds one step to both sides and compares ids, gates, cache trace and outputs.

    Where two of the oracle's logits are closer than NEAR_TIE and the library therefore picked a
    different (equally defensible) set, or the same set with two ranks swapped, the difference is
    counted and the oracle is re-run for that (layer, sequence) with the library's list so that
    later cache states stay comparable.
    """

    def __init__(self, wl, oracle, torch, device="cuda:0"):
        self.wl, self.o, self.torch = wl, oracle, torch
        s = wl.shape
        self.L, self.B, self.K, self.H = s.n_layers, s.batch, s.top_k, s.hidden
        self.d_in = torch.empty((self.L, self.B, self.H), dtype=torch.float32, device=device)
        self.d_out = torch.empty_like(self.d_in)
        self.d_ids = torch.empty((self.L, self.B, self.K), dtype=torch.int32, device=device)
        self.d_g = torch.empty((self.L, self.B, self.K), dtype=torch.float32, device=device)
        self.near_ties = 0              # = boundary flips + rank swaps
        self.boundary_flips = 0         # selected set differs across a rank-K / rank-K+1 gap below NEAR_TIE
        self.rank_swaps = 0             # same set, two near-tied ranks exchanged
        self.max_out_err = 0.0
        self.max_gate_err = 0.0

    def _count_tie(self, kind):
        self.near_ties += 1
        if kind == "boundary":
            self.boundary_flips += 1
        else:
            self.rank_swaps += 1

    def tie_report(self):
        return f"near ties {self.near_ties} (boundary flips {self.boundary_flips}, rank swaps {self.rank_swaps})"

    def gpu_step(self, h, host_api=False):
        t = self.torch
        if host_api:
            out = np.empty((self.L, self.B, self.H), np.float32)
            ids = np.empty((self.L, self.B, self.K), np.int32)
            g = np.empty((self.L, self.B, self.K), np.float32)
            self.wl.stack.decode_step_host(np.ascontiguousarray(h), out, ids, g)
            return ids, g, out
        self.d_in.copy_(t.from_numpy(np.ascontiguousarray(h)))
        self.wl.stack.decode_step(self.d_in, self.d_out, self.d_ids, self.d_g)
        t.cuda.synchronize()
        return self.d_ids.cpu().numpy(), self.d_g.cpu().numpy(), self.d_out.cpu().numpy()

    def step(self, h, ffn="selected", ffn_layers=None, host_api=False, check_trace=True):
        ids, g, out = self.gpu_step(h, host_api)
        return self.compare(h, ids, g, out, ffn, ffn_layers, check_trace)

    def compare(self, h, ids, g, out, ffn="selected", ffn_layers=None, check_trace=True):
        """Sets what the library returned for the layer inputs `h` beside the oracle's step on them."""
        r = self.oracle_step(h, ids, ffn, ffn_layers)
        self.check_against(r, g, out, ffn, ffn_layers, check_trace)
        return r, (ids, g, out)

    def oracle_step(self, h, ids, ffn="selected", ffn_layers=None):
        """The oracle's step on `h`, given only the ids the library selected (needed beforehand to find
        near-ties): selected lists are compared here, everything else in check_against."""
        # First pass of the oracle on a copy of nothing: we need margins before committing,
        # so route without touching state.
        override = {}
        for l in range(self.L):
            for b in range(self.B):
                o_ids, _, margin, z, _ = self.o.route(l, h[l, b])
                kind = near_tie_kind(z, o_ids, ids[l, b])
                assert kind is not None, (
                    f"ids differ at layer {l} seq {b} beyond near-ties (boundary margin {margin}): "
                    f"{[int(e) for e in o_ids]} vs {[int(e) for e in ids[l, b]]}")
                if kind != "same":
                    self._count_tie(kind)
                    override[(l, b)] = [int(e) for e in ids[l, b]]
        r = self.o.step(h, ffn=ffn, id_override=override or None, ffn_layers=ffn_layers)
        assert np.array_equal(r["ids"], ids)
        return r

    def check_against(self, r, g, out, ffn="selected", ffn_layers=None, check_trace=True):
        """Gate weights, cache trace, reuse mass and outputs of the library's last step against the
        oracle's result `r` for the same step."""
        ge = float(np.max(np.abs(r["gates"] - g) / np.maximum(np.abs(r["gates"]), 1e-30)))
        self.max_gate_err = max(self.max_gate_err, ge)
        assert ge <= 1e-4, f"gate weights off by {ge}"
        if check_trace:
            tr = self.wl.stack.last_step_trace()
            for l in range(self.L):
                n = len(r["requests"][l])
                assert tr["n_unique"][l] == n
                assert list(tr["requests"][l][:n]) == r["requests"][l]
                assert [bool(x) for x in tr["hit"][l][:n]] == r["hit"][l]
                assert list(tr["slot"][l][:n]) == r["slot"][l]
                assert list(tr["evicted"][l][:n]) == r["evicted"][l]
        _, _, last_mass = self.wl.stack.reuse_mass(-1, want_last=True)
        assert np.allclose(last_mass, r["mass"].reshape(-1), atol=2e-6), "reuse mass differs"
        if ffn is not None:
            tol = TOL[self.wl.shape.weight_dtype]
            for l in (range(self.L) if ffn_layers is None else ffn_layers):
                e = rel_err(out[l], r["out"][l])
                self.max_out_err = max(self.max_out_err, e)
                assert e <= tol, f"layer {l}: output error {e} > {tol}"

    def step_overlapped(self, h, ffn=None, ffn_layers=None):
        """Same checks as step(), with the oracle's share of the work done while the GPU is still busy
        with the step: the selected ids and gate weights are final when remoe_decode_step returns (the
        call waits for the routing kernels), so they are read on a second stream and the oracle steps on
        the host while the library's fetches and expert kernels run.  For long host-link-bound runs."""
        t = self.torch
        if not hasattr(self, "side"):
            self.side = t.cuda.Stream()
        self.d_in.copy_(t.from_numpy(np.ascontiguousarray(h)))
        self.wl.stack.decode_step(self.d_in, self.d_out, self.d_ids, self.d_g)
        with t.cuda.stream(self.side):
            ids = self.d_ids.cpu().numpy()
            g = self.d_g.cpu().numpy()
        r = self.oracle_step(h, ids, ffn, ffn_layers)
        t.cuda.synchronize()
        out = self.d_out.cpu().numpy() if ffn is not None else None
        self.check_against(r, g, out, ffn, ffn_layers)
        return r, (ids, g, out)

    def step_chained_batched(self, h0):
        """One chained step of a batched stack (h0: [B, H]), checked layer by layer: with bf16 MMA
        operands the residual stream drifts from an fp64 one by about 1e-3, enough to flip a top-K
        choice far from any tie, so an end-to-end comparison of ids would not be meaningful.  Instead
        the library's own residual stream h_0 .. h_L is taken as given: every layer's routing, cache
        trace and MoE output must match the oracle run on x_l = rmsnorm(h_l) (ids exact, outputs within
        tolerance), where the library's layer output is read off as h_{l+1} - h_l."""
        t = self.torch
        L, B, H = self.L, self.B, self.H
        dev = self.d_in.device
        d_h0 = t.from_numpy(np.ascontiguousarray(h0, dtype=np.float32).reshape(B, H)).to(dev)
        d_fin = t.empty((B, H), dtype=t.float32, device=dev)
        d_lin = t.empty((L, B, H), dtype=t.float32, device=dev)
        self.wl.stack.decode_step_chained(d_h0, d_fin, d_lin, self.d_ids, self.d_g)
        t.cuda.synchronize()
        hs = np.concatenate([d_lin.cpu().numpy(), d_fin.cpu().numpy()[None]]).astype(np.float64)   # [L + 1, B, H]
        assert np.array_equal(hs[0].astype(np.float32), np.asarray(h0, dtype=np.float32).reshape(B, H))
        x = hs[:L] / np.sqrt(np.mean(hs[:L] * hs[:L], axis=-1, keepdims=True) + 1e-6)
        out = hs[1:] - hs[:L]
        return self.compare(x, self.d_ids.cpu().numpy(), self.d_g.cpu().numpy(), out)

    def step_chained(self, h0):
        """One chained step (h_{l+1} = h_l + MoE_l(h_l)) on both sides.  A near-tie at one layer
        changes the inputs of the layers below it, so the oracle is first run on a copy to find
        such positions, then for real with the library's ids forced there."""
        import copy
        t = self.torch
        L, H, K = self.L, self.H, self.K
        d_h0 = t.from_numpy(np.ascontiguousarray(h0, dtype=np.float32).reshape(H)).to(self.d_in.device)
        d_fin = t.empty(H, dtype=t.float32, device=d_h0.device)
        d_lin = t.empty((L, H), dtype=t.float32, device=d_h0.device)
        self.wl.stack.decode_step_chained(d_h0, d_fin, d_lin, self.d_ids, self.d_g)
        t.cuda.synchronize()
        ids = self.d_ids.cpu().numpy()
        override = {}
        for _ in range(L + 1):
            trial = copy.deepcopy(self.o).step(np.asarray(h0).reshape(1, H), ffn="selected", chained=True,
                                               id_override=override or None)
            bad = [l for l in range(L) if list(trial["ids"][l, 0]) != list(ids[l, 0])]
            if not bad:
                break
            l = bad[0]
            kind = near_tie_kind(trial["logits"][l, 0], trial["ids"][l, 0], ids[l, 0])
            assert kind is not None, (
                f"chained ids differ at layer {l} beyond near-ties, boundary margin {trial['margin'][l, 0]}")
            self._count_tie(kind)
            override[(l, 0)] = [int(e) for e in ids[l, 0]]
        r = self.o.step(np.asarray(h0).reshape(1, H), ffn="selected", chained=True, id_override=override or None)
        assert np.array_equal(r["ids"], ids)
        tol = TOL[self.wl.shape.weight_dtype]
        e_fin = rel_err(d_fin.cpu().numpy(), r["final"][0])
        e_lin = rel_err(d_lin.cpu().numpy(), r["layer_inputs"][:, 0])
        self.max_out_err = max(self.max_out_err, e_fin, e_lin)
        assert e_fin <= tol and e_lin <= tol, (e_fin, e_lin)
        tr = self.wl.stack.last_step_trace()
        l = L - 1                                   # the trace block holds the last layer's round trip
        assert list(tr["requests"][l][:K]) == r["requests"][l] and list(tr["slot"][l][:K]) == r["slot"][l]
        return r

    def check_directory(self):
        """The library's directory of every layer against the oracle's cache object: which expert sits in
        which slot, the slots' places in the touch order and their use counts (the state C_{t+1} itself, not
        only the trace that led to it)."""
        for l in range(self.L):
            eos, stamp, freq = self.wl.stack.cache_snapshot(l)
            c = self.o.caches[l]
            assert list(eos) == c.expert_of_slot, f"layer {l}: slot contents differ"
            assert [int(x) for x in stamp] == c.stamp, f"layer {l}: touch order differs"
            occupied = [s for s, e in enumerate(c.expert_of_slot) if e >= 0]
            assert [int(freq[s]) for s in occupied] == [c.freq[s] for s in occupied], f"layer {l}: use counts differ"

    def check_counters(self):
        self.check_directory()
        st = self.wl.stack
        o = self.o
        tot = st.cache_stats(-1)
        assert tot["tok_hits"] == sum(o.tok_hits) and tot["tok_misses"] == sum(o.tok_misses)
        assert tot["uniq_hits"] == sum(o.uniq_hits) and tot["uniq_misses"] == sum(o.uniq_misses)
        assert tot["steps"] == o.steps
        assert tot["h2d_bytes"] == sum(o.uniq_misses) * synth.expert_block_bytes(self.wl.shape)
        for l in range(self.L):
            c = st.cache_stats(l)
            assert (c["tok_hits"], c["tok_misses"], c["uniq_hits"], c["uniq_misses"]) == (
                o.tok_hits[l], o.tok_misses[l], o.uniq_hits[l], o.uniq_misses[l])
            ov, pairs = st.reuse_stats(l)
            assert (ov, pairs) == (o.overlap_sum[l], o.pairs_counted[l])
        ov, pairs = st.reuse_stats(-1)
        assert (ov, pairs) == (sum(o.overlap_sum), sum(o.pairs_counted))
        # reporting: reuse mass (Eq. 2), per-step aggregates and the TPOT proxy (App. E.2.6)
        from paper_2605_27081_b200 import binding as B
        m, p = st.reuse_mass(-1)
        assert p == sum(o.pairs_counted) and abs(m - sum(o.mass_sum)) <= 1e-5 * max(1.0, p)
        # expert load: counts exact; entropy and CV are the same double arithmetic on equal integers
        counts, ent, cv, seen = st.expert_load(-1)
        assert (counts.astype(np.int64) == np.asarray(o.load, dtype=np.int64)).all()
        assert abs(ent - o.routing_entropy()) <= 1e-12 and abs(cv - o.routing_cv()) <= 1e-12
        assert seen == int(o.experts_visited())
        c0, ent0, cv0, seen0 = st.expert_load(0)
        assert (c0.astype(np.int64) == np.asarray(o.load[0])).all() and seen0 == o.experts_visited(0)
        assert abs(ent0 - o.routing_entropy(0)) <= 1e-12 and abs(cv0 - o.routing_cv(0)) <= 1e-12
        um, th = st.step_history()
        assert list(um) == o.hist_umiss and list(th) == o.hist_tok_hits
        if len(um):
            eb = synth.expert_block_bytes(self.wl.shape)
            rc, io, pct = B.remoe_tpot_proxy(um, eb, 4.0, self.B, 12.5)
            t_ref, pct_ref = orc.tpot_proxy(um, eb, 4.0, self.B, 12.5)
            assert rc == 0 and np.allclose(io, orc.io_ms_step(um, eb, 4.0), rtol=1e-12)
            assert np.allclose(pct, pct_ref, rtol=1e-12)
