"""CPU oracle for the bounded-cache MoE decode step (TEST INFRASTRUCTURE ONLY).

A plain, slow, fp64 restatement of what one decode step computes: router logits,
softmax, top-K selection, resolution of the requested experts against a per-layer
cache of C slots with LRU replacement, the SwiGLU expert outputs combined with the
gate weights (plus always-resident shared experts), and the step-to-step reuse
statistic.  It exists so that tests, the smoke check and the benchmark's CPU-baseline
leg have something independent to compare the CUDA library against.  It shares no code
with that library, imports nothing from it, and must never be imported by it.

What follows the paper (ReMoE, "Boosting Expert Reuse through Router Fine-Tuning ..."):

* routing  P_t = Softmax(h_t^T theta_gate), E_t = Top-K(P_t), shared experts always
  active and excluded from P_t                                   -- Sec. 3.1
* cache state C_t "before serving step t", |C_t| <= C, fetch count
  N_fetch(t) = |E_t \\ C_t|                                       -- App. A.1, Eq. (fetch_def)
* serve-and-admit update, step atomicity, E_t subset of C_{t+1}  -- App. A.2, Assumption 2
* LRU keeps the most recently used distinct experts              -- App. A.5
* token-level and unique-level hits/misses, R, U = Unique(R)     -- App. E.2.2-E.2.3
* aggregates #uMiss, uHR, tHR                                    -- App. E.2.4
* IR_t = |E_t n E_{t-1}| / K, EOR = mean_{t>=2} IR_t             -- Sec. 3.2, Eq. (1)

Where the paper is silent this file takes the following readings (each is also a
documented property of the CUDA library, so the two can be compared):

* Top-K is taken on the logits z (exp is monotone); equal logits go to the lower index;
  the selected list is ordered by (z descending, index ascending).
* Gate weight of a selected expert is P_e, or P_e / sum_{j in E} P_j with `renorm_topk`.
* An expert is SwiGLU without biases: y = W_down (silu(W_gate x) * (W_up x)),
  silu(v) = v / (1 + exp(-v)).  Shared experts add sum_s scale * y_s with scale = 1, or
  sigmoid(w_sg . x) when `shared_gate` is set.
* Cache update is two-phase: every request is classified against C_t first; then hits
  are touched in request order, then misses are inserted in request order, each taking
  the lowest-index empty slot if one exists and otherwise the slot with the oldest touch
  among occupants that are not part of this step's request (step atomicity); only when
  every slot holds one of this step's experts -- more distinct requests than slots -- does
  the oldest touch among all slots go (later misses displace this step's earlier entries).
* Each layer has its own input stream: out[l] = MoE_l(h[l]); layers do not feed each other.

Parity pins (tests/test_oracle_*.py): softmax against closed forms and scipy, top-K against the
counting definition and constructed ties, LRU/FIFO/LFU against hand-worked slot traces and LRU
against the set characterisation "the C most recently used distinct experts" recomputed from
the whole history, the exact identity misses(t) = K - |E_t n E_{t-1}| when C = K (App. A.3
"Tightness"), both fetch bounds, Belady against exhaustive search, counters against their
totals and against the uHR / #uMiss table the paper prints (App. F.1), the TPOT proxy against
the slope of the paper's TPOT table, the load entropy and CV against closed forms and the
(entropy, CV) pairs the paper prints, the FFN against a hand example and a library matmul in the
N = K = 1 case, dense-and-mask against selected-only, linearity in the gate weights, the
chained mode against its telescoping sum and hand-run one-layer stacks.  Every function has at
least one such pin, so none is "parity unpinned"; but the paper prints no worked numeric
example of a layer output, so absolute float outputs rest on those special cases and library
routines alone.
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


# ----------------------------------------------------------------------------- routing

def router_logits(w_router, h):
    """z_i = sum_j W_r[i, j] h[j]  (Sec. 3.1: h_t^T theta_gate), fp64."""
    return np.asarray(w_router, dtype=F64) @ np.asarray(h, dtype=F64)


def softmax(z):
    """P = exp(z - max z) / sum exp(z - max z)  (Sec. 3.1)."""
    z = np.asarray(z, dtype=F64)
    e = np.exp(z - np.max(z))
    return e / np.sum(e)


def topk_select(z, k):
    """First k indices of a full sort by (z descending, index ascending).

    Returns (ids [k] int64, margin) with margin = z_(k) - z_(k+1), the gap between the
    last selected and the first rejected logit (inf when k == len(z)).
    """
    z = np.asarray(z, dtype=F64)
    n = z.shape[0]
    order = sorted(range(n), key=lambda i: (-z[i], i))
    ids = np.array(order[:k], dtype=np.int64)
    margin = float(z[order[k - 1]] - z[order[k]]) if k < n else float("inf")
    return ids, margin


def gate_weights(p, ids, renorm):
    """g_e = P_e for e in E, divided by their sum when `renorm` is set."""
    g = np.asarray(p, dtype=F64)[np.asarray(ids)]
    if renorm:
        g = g / np.sum(g)
    return g


def unique_in_order(r):
    """U = Unique(R), first-occurrence order (App. E.2.3)."""
    seen, out = set(), []
    for e in r:
        e = int(e)
        if e not in seen:
            seen.add(e)
            out.append(e)
    return out


def reuse_mass(p_t, e_prev, k):
    """m_t = (1/K) sum_{j in E_{t-1}} P_t^(j), the reuse mass (Eq. 2)."""
    p_t = np.asarray(p_t, dtype=F64)
    return float(sum(p_t[int(j)] for j in e_prev) / k)


def io_ms_step(umiss, expert_bytes, bandwidth_gbps):
    """IO_ms_step = #uMiss * expert_bytes / bandwidth * 1000, bandwidth in 1e9 bytes/s (App. E.2.6)."""
    return np.asarray(umiss, dtype=F64) * float(expert_bytes) / (float(bandwidth_gbps) * 1e9) * 1000.0


def tpot_proxy(umiss, expert_bytes, bandwidth_gbps, batch=1, tpot_compute_ms=0.0):
    """TPOT ~ TPOT_compute + IO_step / B per step (App. F.1), and its P50/P95/P99 over the steps
    (linear interpolation between order statistics; the paper does not say which rule it uses)."""
    tpot = tpot_compute_ms + io_ms_step(umiss, expert_bytes, bandwidth_gbps) / batch
    srt = sorted(float(x) for x in tpot)
    out = []
    for q in (0.50, 0.95, 0.99):
        pos = q * (len(srt) - 1)
        lo = int(pos)
        hi = min(lo + 1, len(srt) - 1)
        out.append(srt[lo] + (pos - lo) * (srt[hi] - srt[lo]))
    return tpot, out


def load_entropy(counts):
    """Normalised routing entropy: H(p) / log N of the empirical load distribution p_e = n_e / sum n,
    n_e = how often expert e was selected (Sec. 4.4 "Routing imbalance"; Sec. 5.2, table of routing
    metrics).  The
    paper prints the numbers without a formula; this reading is the one its own (entropy, CV) pairs
    satisfy: near balance H / log N = 1 - CV^2 / (2 log N) + O(CV^3).  1 = perfectly even load."""
    n = np.asarray(counts, dtype=F64)
    tot = float(n.sum())
    if tot <= 0.0 or n.size < 2:
        return 1.0
    h = 0.0
    for v in n:                                   # 0 log 0 = 0
        if v > 0.0:
            q = float(v) / tot
            h -= q * np.log(q)
    return float(h / np.log(float(n.size)))


def load_cv(counts):
    """Load-balance coefficient of variation: population standard deviation of the per-expert
    selection counts over their mean (Sec. 4.4 "Routing imbalance"; Sec. 5.2).  0 = perfectly even load."""
    n = np.asarray(counts, dtype=F64)
    mean = float(n.sum()) / n.size
    if mean <= 0.0:
        return 0.0
    var = float(((n - mean) ** 2).sum()) / n.size
    return float(np.sqrt(var) / mean)


def reuse_overlap(e_t, e_prev):
    """|E_t n E_{t-1}|, the numerator of IR_t (Eq. 1)."""
    return len(set(int(x) for x in e_t) & set(int(x) for x in e_prev))


# ------------------------------------------------------------------------------- cache

class SlotCache:
    """One layer's expert cache: C slots, each holding one expert id or nothing.

    `serve(requests)` takes the step's distinct requests in order and returns, per
    request, (hit, slot, evicted_id).  Hits and misses are decided against the state
    held before the call (App. A.1); the update then follows the two-phase rule in
    the file header.  `policy` is "lru" (default), "fifo" or "lfu".
    """

    def __init__(self, capacity, policy="lru"):
        self.capacity = int(capacity)
        self.policy = policy
        self.expert_of_slot = [-1] * self.capacity
        self.stamp = [0] * self.capacity      # lru: last touch; fifo: insertion time
        self.freq = [0] * self.capacity       # lfu only
        self.clock = 0

    def resident(self):
        return set(e for e in self.expert_of_slot if e >= 0)

    def slot_of(self, expert):
        for s, e in enumerate(self.expert_of_slot):
            if e == expert:
                return s
        return -1

    def _victim(self, in_use):
        for s, e in enumerate(self.expert_of_slot):
            if e < 0:
                return s
        # Step atomicity (App. A.2): experts of the current request are not candidates
        # while any other occupant exists.  (Under LRU with no more requests than slots
        # this never changes the choice: the step's experts carry the newest touches.)
        cand = [s for s in range(self.capacity) if self.expert_of_slot[s] not in in_use]
        if not cand:
            cand = list(range(self.capacity))
        if self.policy == "lfu":
            key = {s: (self.freq[s], self.stamp[s]) for s in cand}
        else:
            key = {s: self.stamp[s] for s in cand}
        best = cand[0]
        for s in cand[1:]:
            if key[s] < key[best]:
                best = s
        return best

    def serve(self, requests):
        requests = [int(e) for e in requests]
        before = [self.slot_of(e) for e in requests]       # classification against C_t
        hit = [s >= 0 for s in before]
        slot = list(before)
        evicted = [-1] * len(requests)
        in_use = set(requests)
        for i, e in enumerate(requests):                   # phase 1: touch hits in order
            if hit[i]:
                self.clock += 1
                s = before[i]
                if self.policy != "fifo":
                    self.stamp[s] = self.clock
                self.freq[s] += 1
        for i, e in enumerate(requests):                   # phase 2: admit misses in order
            if not hit[i]:
                self.clock += 1
                s = self._victim(in_use)
                evicted[i] = self.expert_of_slot[s]
                self.expert_of_slot[s] = e
                self.stamp[s] = self.clock
                self.freq[s] = 1
                slot[i] = s
        return hit, slot, evicted


def belady_min_misses(requests_per_step, capacity):
    """Misses of the offline-optimal policy (evict the resident expert whose next use is
    farthest in the future) on one layer's trace; each step's distinct requests are
    served together and are never evicted within their own step.  Analysis only."""
    steps = [unique_in_order(r) for r in requests_per_step]
    next_use = []
    last = {}
    for t in range(len(steps) - 1, -1, -1):
        nu = {}
        for e in steps[t]:
            nu[e] = last.get(e, float("inf"))
        for e in steps[t]:
            last[e] = t
        next_use.append(nu)
    next_use.reverse()
    resident, nxt, misses = set(), {}, 0
    for t, req in enumerate(steps):
        for e in req:
            if e not in resident:
                misses += 1
        for e in req:
            nxt[e] = next_use[t][e]
        pinned = set(req)
        resident |= pinned
        while len(resident) > capacity:
            cand = [e for e in resident if e not in pinned] or list(resident)
            victim = max(cand, key=lambda e: (nxt[e], e))
            resident.discard(victim)
    return misses


# --------------------------------------------------------------------------------- FFN

def silu(v):
    v = np.asarray(v, dtype=F64)
    return v / (1.0 + np.exp(-v))


def swiglu_expert(w_gate, w_up, w_down, x):
    """y = W_down (silu(W_gate x) * (W_up x)); W_gate, W_up: [I, H]; W_down: [H, I]."""
    x = np.asarray(x, dtype=F64)
    a = silu(np.asarray(w_gate, dtype=F64) @ x) * (np.asarray(w_up, dtype=F64) @ x)
    return np.asarray(w_down, dtype=F64) @ a


def moe_output(x, ids, gates, n_routed, expert_weights, shared_weights=(), shared_scale=1.0,
               mode="dense"):
    """out = sum_e m_e g_e y_e(x) + sum_s shared_scale * y_s(x), e ascending.

    `expert_weights(e)` returns (W_gate, W_up, W_down) of routed expert e.  In "dense"
    mode every routed expert is evaluated and masked by m_e = [e in E]; "selected" skips
    the experts with m_e = 0 and is otherwise the same sum in the same order.
    """
    x = np.asarray(x, dtype=F64)
    g_of = {int(e): float(g) for e, g in zip(ids, gates)}
    out = np.zeros(x.shape[0], dtype=F64)
    for e in range(n_routed):
        m = 1.0 if e in g_of else 0.0
        if mode == "selected" and m == 0.0:
            continue
        y = swiglu_expert(*expert_weights(e), x)
        out = out + (m * g_of.get(e, 0.0)) * y
    for w in shared_weights:
        out = out + shared_scale * swiglu_expert(*w, x)
    return out


def sigmoid(v):
    return 1.0 / (1.0 + np.exp(-float(v)))


# ------------------------------------------------------------------------------- stack

class OracleStack:
    """L independent MoE layers, each with its own cache, stepped one token at a time.

    shape: any object with n_layers, hidden, n_routed, top_k, n_shared, shared_gate,
    renorm_topk, batch.  `routers[l]` is [N, H]; `shared_gates[l]` is [H] or None;
    `expert_weights(l, e)` / `shared_weights(l, s)` return (W_gate, W_up, W_down) as
    float arrays holding the exact stored values (bf16 already widened).
    """

    def __init__(self, shape, cache_slots, routers, expert_weights=None, shared_weights=None,
                 shared_gates=None, policy="lru", reroute_beta=0.0):
        self.s = shape
        self.C = int(cache_slots)
        self.routers = [np.asarray(w, dtype=F64) for w in routers]
        self.shared_gates = shared_gates
        self.expert_weights = expert_weights
        self.shared_weights = shared_weights
        self.policy = policy
        self.reroute_beta = float(reroute_beta)
        self.reset()

    def reset(self):
        """Request-isolated cold start (Sec. 3): empty caches, no previous selection."""
        L, B = self.s.n_layers, self.s.batch
        self.caches = [SlotCache(self.C, self.policy) for _ in range(L)]
        self.prev = [[None] * B for _ in range(L)]
        self.tok_hits = [0] * L
        self.tok_misses = [0] * L
        self.uniq_hits = [0] * L
        self.uniq_misses = [0] * L
        self.overlap_sum = [0] * L
        self.pairs_counted = [0] * L
        self.mass_sum = [0.0] * L
        self.load = [[0] * self.s.n_routed for _ in range(L)]   # selections per expert (token level)
        self.hist_umiss = []          # per step, summed over layers (App. E.2.6)
        self.hist_tok_hits = []
        self.steps = 0

    def route(self, l, h_lb, override=None):
        """One (layer, sequence): logits, softmax, top-K, gate weights."""
        s = self.s
        z = router_logits(self.routers[l], h_lb)
        p = softmax(z)
        score = z
        if self.reroute_beta != 0.0:
            # cache-aware rerouting (App. F.2): bonus on the pre-Top-K scores of experts
            # resident before the step; the gate weights still come from P.
            bonus = np.zeros_like(z)
            for e in self.caches[l].resident():
                bonus[e] = self.reroute_beta
            score = z + bonus
        ids, margin = topk_select(score, s.top_k)
        if override is not None:
            ids = np.asarray(override, dtype=np.int64)
        g = gate_weights(p, ids, s.renorm_topk)
        return ids, g, margin, z, p

    def step(self, h, ffn="selected", id_override=None, ffn_layers=None, chained=False):
        """Advance every layer by one token.  h: [L, B, H].

        chained=True: h is [B, H], the input of layer 0, and the layers feed each other through
        a pre-norm residual connection, x_l = h_l / sqrt(mean(h_l^2) + 1e-6) and
        h_{l+1} = h_l + MoE_l(x_l) (how MoE layers sit in a decoder; the paper's analysis treats
        each layer on its own).  The result then also carries "layer_inputs" [L, B, H] (the
        residual stream h_l) and "final" [B, H]; `ffn` must not be None.

        ffn: "dense", "selected" or None (integer parts only).  `ffn_layers` restricts the
        floating-point FFN to some layers.  `id_override[(l, b)]` forces the selected ids
        of one (layer, sequence) -- used only to keep cache traces comparable after a
        near-tie (the caller checks the margin).
        """
        s = self.s
        L, B, K = s.n_layers, s.batch, s.top_k
        h = np.asarray(h)
        res = dict(
            ids=np.zeros((L, B, K), np.int64), gates=np.zeros((L, B, K), F64),
            margin=np.zeros((L, B), F64), logits=np.zeros((L, B, s.n_routed), F64),
            overlap=np.full((L, B), -1, np.int64),
            mass=np.full((L, B), -1.0, F64),
            requests=[], hit=[], slot=[], evicted=[], tok_hits=[],
            out=None if ffn is None else np.zeros((L, B, s.hidden), F64),
            shared_scale=np.ones((L, B), F64))
        if chained:
            cur = np.asarray(h, dtype=F64).reshape(B, s.hidden).copy()
            res["layer_inputs"] = np.zeros((L, B, s.hidden), F64)
        for l in range(L):
            if chained:
                res["layer_inputs"][l] = cur
                hl = cur / np.sqrt(np.mean(cur * cur, axis=1, keepdims=True) + 1e-6)
            else:
                hl = h[l]
            flat = []
            for b in range(B):
                ov = None if id_override is None else id_override.get((l, b))
                ids, g, margin, z, p = self.route(l, hl[b], ov)
                res["ids"][l, b], res["gates"][l, b], res["margin"][l, b] = ids, g, margin
                res["logits"][l, b] = z
                flat.extend(int(e) for e in ids)
                for e in ids:
                    self.load[l][int(e)] += 1
                if self.prev[l][b] is not None:                       # Eq. (1), t >= 2
                    ov_n = reuse_overlap(ids, self.prev[l][b])
                    res["overlap"][l, b] = ov_n
                    self.overlap_sum[l] += ov_n
                    self.pairs_counted[l] += 1
                    res["mass"][l, b] = reuse_mass(p, self.prev[l][b], K)          # Eq. (2)
                    self.mass_sum[l] += res["mass"][l, b]
                self.prev[l][b] = [int(e) for e in ids]
                if s.shared_gate:
                    res["shared_scale"][l, b] = sigmoid(
                        np.asarray(self.shared_gates[l], dtype=F64) @ np.asarray(hl[b], dtype=F64))
            cache = self.caches[l]
            before = cache.resident()                                  # C_t
            th = sum(1 for e in flat if e in before)                   # token level, App. E.2.3
            self.tok_hits[l] += th
            res["tok_hits"].append(th)
            self.tok_misses[l] += len(flat) - th
            req = unique_in_order(flat)                                # U
            hit, slot, evicted = cache.serve(req)
            self.uniq_hits[l] += sum(hit)
            self.uniq_misses[l] += len(req) - sum(hit)
            res["requests"].append(req)
            res["hit"].append(hit)
            res["slot"].append(slot)
            res["evicted"].append(evicted)
            if ffn is not None and (ffn_layers is None or l in ffn_layers):
                shared = [self.shared_weights(l, i) for i in range(s.n_shared)]
                for b in range(B):
                    res["out"][l, b] = moe_output(
                        hl[b], res["ids"][l, b], res["gates"][l, b], s.n_routed,
                        lambda e, l=l: self.expert_weights(l, e), shared,
                        res["shared_scale"][l, b], mode=ffn)
            if chained:
                cur = cur + res["out"][l]
        if chained:
            res["final"] = cur
        self.hist_umiss.append(sum(len(hh) - sum(hh) for hh in res["hit"]))
        self.hist_tok_hits.append(sum(res["tok_hits"]))
        self.steps += 1
        return res

    # aggregates (App. E.2.4)
    def uhr(self, layer=None):
        ls = range(self.s.n_layers) if layer is None else [layer]
        h = sum(self.uniq_hits[l] for l in ls)
        m = sum(self.uniq_misses[l] for l in ls)
        return h / (h + m) if h + m else 0.0

    def thr(self, layer=None):
        ls = range(self.s.n_layers) if layer is None else [layer]
        h = sum(self.tok_hits[l] for l in ls)
        m = sum(self.tok_misses[l] for l in ls)
        return h / (h + m) if h + m else 0.0

    def routing_entropy(self, layer=None):
        """Normalised load entropy of one layer, or its mean over the layers."""
        ls = range(self.s.n_layers) if layer is None else [layer]
        return sum(load_entropy(self.load[l]) for l in ls) / len(ls)

    def routing_cv(self, layer=None):
        """Load-balance CV of one layer, or its mean over the layers."""
        ls = range(self.s.n_layers) if layer is None else [layer]
        return sum(load_cv(self.load[l]) for l in ls) / len(ls)

    def experts_visited(self, layer=None):
        """Distinct experts selected at least once in one layer, or the mean over the layers."""
        ls = range(self.s.n_layers) if layer is None else [layer]
        return sum(sum(1 for v in self.load[l] if v > 0) for l in ls) / len(ls)

    def eor(self, layer=None):
        ls = range(self.s.n_layers) if layer is None else [layer]
        num = sum(self.overlap_sum[l] for l in ls)
        den = sum(self.pairs_counted[l] for l in ls) * self.s.top_k
        return num / den if den else 0.0
