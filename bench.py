#!/usr/bin/env python
"""Decode-throughput benchmark of the bounded-cache MoE decode step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--rho R] [--impl ours|reference]

A "step" is one decode step: one token (or one token of each of B sequences) through all MoE layers of
a stack, driven by seeded AR(1) hidden states.  The line's `value` is measured on the
DeepSeek-V2-Lite-shaped batch-1 stack (26 layers, hidden 2048, 64 routed experts top-6 + 2 shared,
intermediate 1408, bf16 weights, 16 cache slots per layer, LRU) from device-resident inputs: cold cache,
W warm-up steps, then exactly K timed steps; the same steps are then repeated through host buffers
(`e2e`).  Both are run `--repeats` times on identical inputs and the median repeat is reported with the
minimum and maximum.  One JSON line is printed by rank 0.  With N > 1 every rank runs an independent
replica (the path has no exchange step); the time is the maximum over ranks and the value the sum of
tokens.  The other workloads (`other_workloads` in the line) are short runs of the same protocol.
"""
from __future__ import annotations

import argparse
import copy
import json
import os
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import synth  # noqa: E402

WORKLOAD = "dsv2lite"
NOMINAL_HBM_GBS = 8000.0
COLD_STEPS = 32
# DRAM bytes (read + write) per algorithmic byte of a resident-phase launch of the expert kernel, from the
# profiler captures of that kernel on a shallower stack of the same layer shape (traffic grows in proportion
# to the blocks streamed).  Keyed by (workload, kernel); valid only for the kernel it was taken on, so an
# entry is dropped (None) when that kernel changes.
TRAFFIC_RATIO = {
    ("dsv2lite", "ffn_stream_kernel<bf16,2048>"): 1.010,
    ("dsv2lite_fp8", "ffn_stream_kernel<fp8_e4m3,2048>"): 1.029,
    ("dsv2lite_b32", "ffn_batched_tc_kernel<2048>"): 1.062,      # includes the second pass over the shared experts
}
DTYPE_NAME = {0: "f32", 1: "bf16", 2: "fp8_e4m3", 3: "int4_g32"}      # weight storage; accumulation is always f32
CLOCK_QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
               "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
               "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")


_T0 = time.perf_counter()


def note(msg):
    """Progress line on stderr (the JSON line on stdout stays alone)."""
    print(f"[bench {time.perf_counter() - _T0:7.1f}s] {msg}", file=sys.stderr, flush=True)


def metric_name(shape):
    return f"decode tokens/s (batch {shape.batch}, MoE stack)"


def kernel_name(shape):
    """The expert kernel a stack of this shape runs (the library picks it the same way)."""
    if shape.batch == 1:
        return f"ffn_stream_kernel<{DTYPE_NAME[shape.weight_dtype]},{shape.hidden}>"
    tc = shape.inter_routed % 64 == 0 and (shape.n_shared == 0 or shape.inter_shared % 64 == 0)
    if tc and os.environ.get("REMOE_BATCHED_KERNEL") != "mma":
        return f"ffn_batched_tc_kernel<{shape.hidden}>"
    return f"ffn_batched_kernel<{shape.hidden}>"


def measured_peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


class ClockSampler:
    def __init__(self, index):
        self.path = os.path.join("/tmp", f"remoe_clocks_{os.getpid()}.csv")
        self.f = open(self.path, "w")
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--id={index}", f"--query-gpu={CLOCK_QUERY}",
                                       "--format=csv,noheader,nounits", "-lms", "100"],
                                      stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self):
        if self.p is not None:
            self.p.terminate()
            try:
                self.p.wait(timeout=5)
            except Exception:
                self.p.kill()
        self.f.close()
        sm, mx, reasons, power = [], [], set(), []
        try:
            for line in open(self.path):
                c = [x.strip() for x in line.split(",")]
                if len(c) < 9:
                    continue
                try:
                    sm.append(float(c[1])); mx.append(float(c[2])); power.append(float(c[3]))
                except ValueError:
                    continue
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), c[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            os.remove(self.path)
        except Exception:
            pass
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons),
                "samples": len(sm), "power_w_max": float(max(power))}


def merge_clocks(per_repeat):
    got = [c for c in per_repeat if c and c.get("sm_mhz") is not None]
    if not got:
        return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0, "per_repeat_sm_mhz": []}
    return {"sm_mhz": float(np.median([c["sm_mhz"] for c in got])), "sm_max_mhz": max(c["sm_max_mhz"] for c in got),
            "reasons": sorted(set().union(*[set(c["reasons"]) for c in got])),
            "samples": sum(c["samples"] for c in got), "power_w_max": max(c["power_w_max"] for c in got),
            "per_repeat_sm_mhz": [c["sm_mhz"] for c in got]}


# ------------------------------------------------------------------------------- CPU oracle legs

def _blas_threads():
    try:
        from threadpoolctl import threadpool_info
        return max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        return 1


def oracle_sample(shape, cache_slots, seed, rho, layers, steps, warm_steps, mode="selected", threads=None, store=None):
    """Time the CPU oracle, as it stands, on the first `layers` layers for `steps` decode steps after
    `warm_steps` steps that fill its caches (integer parts only).  `threads`: limit of the BLAS pool
    (None = whatever the process has).  Returns (seconds, threads the BLAS pool had)."""
    from oracle import remoe_oracle as orc
    sub = synth.Shape(**{**shape.asdict(), "n_layers": layers})
    routers = [synth.widen(shape, synth.gen_router(seed, shape, l), True) for l in range(layers)]
    gates = [synth.widen(shape, synth.gen_shared_gate(seed, shape, l), True) for l in range(layers)] \
        if shape.shared_gate else None
    blocks = {}

    def ew(l, e):
        if (l, e) not in blocks:
            raw = store(l, e) if store is not None else synth.gen_expert_block(seed, shape, l, e)
            blocks[(l, e)] = synth.widen(shape, raw)
        return synth.expert_matrices(blocks[(l, e)], shape.hidden, shape.inter_routed)

    shared = {(l, i): synth.widen(shape, synth.gen_shared_block(seed, shape, l, i)) for l in range(layers)
              for i in range(shape.n_shared)}

    def sw(l, i):
        return synth.expert_matrices(shared[(l, i)], shape.hidden, shape.inter_shared)

    st = orc.OracleStack(sub, cache_slots, routers, ew, sw, shared_gates=gates)
    hs = synth.HiddenStream(seed, shape, rho)
    hidden = [hs.step()[:layers] for _ in range(warm_steps + steps)]
    # every weight the timed steps touch is widened before the clock starts (the GPU side also starts with
    # its store ready): a dry run of the integer parts tells which
    for t in range(warm_steps + steps):
        r = st.step(hidden[t], ffn=None)
        if t >= warm_steps:
            for l in range(layers):
                for e in (range(shape.n_routed) if mode == "dense" else r["ids"][l].reshape(-1)):
                    ew(l, int(e))
    st.reset()
    for t in range(warm_steps):
        st.step(hidden[t], ffn=None)

    def timed():
        t0 = time.perf_counter()
        for t in range(warm_steps, warm_steps + steps):
            st.step(hidden[t], ffn=mode)
        return time.perf_counter() - t0

    if threads is not None:
        try:
            from threadpoolctl import threadpool_limits
            with threadpool_limits(limits=threads):
                return timed(), threads
        except Exception:
            pass
    return timed(), _blas_threads()


def cpu_baseline_legs(shape, C, seed, rho, store):
    """The oracle on a bounded sample of the headline workload: selected-experts-only on one thread and on
    all host cores (the reported baseline), and dense-and-mask on the tiny configuration in full and on a
    prefix of this one."""
    layers, steps, warm = min(8, shape.n_layers), 8, 8
    affinity = len(os.sched_getaffinity(0))
    dt_all, thr_all = oracle_sample(shape, C, seed, rho, layers, steps, warm, store=store)
    dt_one, _ = oracle_sample(shape, C, seed, rho, min(2, layers), steps, warm, threads=1, store=store)
    per_all = dt_all / steps * shape.n_layers / layers
    per_one = dt_one / steps * shape.n_layers / min(2, layers)
    tiny = synth.config("tiny_fp32")
    dt_tiny, _ = oracle_sample(tiny["shape"], tiny["cache_slots"], tiny["seed"], tiny["rhos"][0], 1, tiny["steps"], 0,
                               mode="dense")
    dt_dense, _ = oracle_sample(shape, C, seed, rho, 1, 8, 0, mode="dense", store=store)
    return {
        "value": shape.batch / per_all, "unit": "tokens/s", "cores": thr_all, "kind": "oracle",
        "sample": (f"steps {warm + 1}..{warm + steps} of the workload (caches warm) over the first {layers} of "
                   f"{shape.n_layers} layers, time scaled by {shape.n_layers}/{layers}; selected-experts-only fp64 "
                   f"oracle, numpy BLAS pool of {thr_all} threads"),
        "host_cores_sched_getaffinity": affinity,
        "one_thread": {"value": shape.batch / per_one, "unit": "tokens/s",
                       "sample": f"same steps over the first {min(2, layers)} layers, BLAS pool limited to 1 thread"},
        "dense_and_mask": {
            "tiny_fp32_full": {"steps": tiny["steps"], "seconds": dt_tiny, "tokens_per_s": tiny["steps"] / dt_tiny},
            "headline_prefix": {"steps": 8, "layers": 1, "seconds": dt_dense,
                                "tokens_per_s_scaled": shape.batch / (dt_dense / 8 * shape.n_layers),
                                "note": "every routed expert evaluated and masked, first 8 steps, first layer, "
                                        f"time scaled by {shape.n_layers}"}},
    }


def run_reference(args, rank, world):
    """The oracle timed on the host cores: each step is one decode step over a sample of layers,
    scaled to the full depth."""
    if rank != 0:
        return
    cfg = synth.config(args.workload)
    shape = cfg["shape"]
    total = args.steps + args.warmup
    layers = int(max(1, min(4, 300 // max(1, total))))
    dt, cores = oracle_sample(shape, cfg["cache_slots"], cfg["seed"], args.rho, layers, args.steps, args.warmup)
    per_step = dt / args.steps * shape.n_layers / layers
    value = shape.batch / per_step
    sample = (f"{args.steps} decode steps (after {args.warmup} cache-warming steps) over the first {layers} of "
              f"{shape.n_layers} layers, time scaled by {shape.n_layers}/{layers}; selected-experts-only fp64 oracle, "
              f"numpy BLAS pool of {cores} threads, {len(os.sched_getaffinity(0))} host cores available")
    line = {
        "impl": "reference", "metric": metric_name(shape), "value": value, "unit": "tokens/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": per_step * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "rho": args.rho, "cache_slots": cfg["cache_slots"], "batch": shape.batch},
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------- GPU legs

class Leg:
    """Device buffers and counters for timed legs on one stack."""

    def __init__(self, torch, wl, stream, shape):
        self.torch, self.wl, self.stream, self.shape = torch, wl, stream, shape
        L, H, K, B = shape.n_layers, shape.hidden, shape.top_k, shape.batch
        self.d_out = torch.empty((L, B, H), dtype=torch.float32, device="cuda")
        self.d_ids = torch.empty((L, B, K), dtype=torch.int32, device="cuda")
        self.d_g = torch.empty((L, B, K), dtype=torch.float32, device="cuda")
        self.out_h = torch.empty((L, B, H), dtype=torch.float32).pin_memory().numpy()
        self.ids_h = torch.empty((L, B, K), dtype=torch.int32).pin_memory().numpy()
        self.g_h = torch.empty((L, B, K), dtype=torch.float32).pin_memory().numpy()

    def snapshot(self):
        st = self.wl.stack
        c = st.cache_stats()
        ov = st.reuse_stats()
        return dict(c, overlap=ov[0], pairs=ov[1], launches=st.launch_count())

    @staticmethod
    def delta(a, b):
        return {k: b[k] - a[k] for k in ("uniq_hits", "uniq_misses", "h2d_bytes", "overlap", "pairs", "launches")}

    def device_steps(self, d_hidden, first, count):
        """`count` decode steps from device-resident inputs; elapsed ms (CUDA events on the stack's stream)."""
        torch = self.torch
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        with torch.cuda.stream(self.stream):
            a.record(self.stream)
            for t in range(first, first + count):
                self.wl.stack.decode_step(d_hidden[t], self.d_out, self.d_ids, self.d_g)
            b.record(self.stream)
        torch.cuda.synchronize()
        return a.elapsed_time(b)

    def host_steps(self, h_hidden, first, count):
        """The same steps through host buffers: inputs copied in, outputs read back, every step."""
        torch = self.torch
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        a.record(self.stream)
        for t in range(first, first + count):
            self.wl.stack.decode_step_host(h_hidden[t], self.out_h, self.ids_h, self.g_h)
        b.record(self.stream)
        torch.cuda.synchronize()
        wall = (time.perf_counter() - t0) * 1e3
        return max(a.elapsed_time(b), wall)


def run_protocol(torch, wl, stream, shape, seed, rho, steps, warmup, repeats, with_e2e, with_cold, local_rank=None,
                 prewarm_iid=0):
    """Per repeat, all from the same hidden states: [cold cache -> COLD_STEPS timed steps]; cold cache -> W
    warm-up steps -> K timed steps from device inputs; [cold cache -> W warm-up steps -> the same K steps
    through host buffers].  Returns the list of per-repeat results."""
    n = max(warmup + steps, COLD_STEPS if with_cold else 0)
    hidden = synth.HiddenStream(seed, shape, rho).take(n)
    h_pinned = torch.from_numpy(hidden).pin_memory()
    d_hidden = h_pinned.to("cuda", non_blocking=False)
    hp = h_pinned.numpy()
    st = wl.stack
    leg = Leg(torch, wl, stream, shape)
    st.set_profiling(False)
    d_pre = None
    if prewarm_iid:
        # independent hidden states touch every expert quickly, so a cache as large as the expert set ends
        # up holding all of them before the measured stream starts
        d_pre = torch.from_numpy(synth.HiddenStream(seed + 1, shape, 0.0).take(prewarm_iid)).to("cuda")

    def fresh():
        st.cache_reset()
        torch.cuda.synchronize()
        if d_pre is not None:
            leg.device_steps(d_pre, 0, prewarm_iid)

    reps = []
    for rep in range(repeats):
        sampler = ClockSampler(local_rank) if local_rank is not None else None
        res = {}
        if with_cold:
            fresh()
            s0 = leg.snapshot()
            ms = leg.device_steps(d_hidden, 0, COLD_STEPS)
            res["cold"] = dict(Leg.delta(s0, leg.snapshot()), ms=ms, steps=COLD_STEPS)
        fresh()
        leg.device_steps(d_hidden, 0, warmup)
        s0 = leg.snapshot()
        st.set_profiling(True)
        res["ms"] = leg.device_steps(d_hidden, warmup, steps)
        res.update(Leg.delta(s0, leg.snapshot()))
        res["kernel_resident"] = st.kernel_time(0)
        res["kernel_miss"] = st.kernel_time(1)
        st.set_profiling(False)
        if with_e2e:
            fresh()
            for t in range(warmup):
                st.decode_step_host(hp[t], leg.out_h, leg.ids_h, leg.g_h)
            s0 = leg.snapshot()
            ms = leg.host_steps(hp, warmup, steps)
            res["e2e"] = dict(Leg.delta(s0, leg.snapshot()), ms=ms, in_bytes=hp[0].nbytes,
                              out_bytes=leg.out_h.nbytes + leg.ids_h.nbytes + leg.g_h.nbytes)
        if sampler is not None:
            res["clocks"] = sampler.stop()
        reps.append(res)
    return reps


def median_rep(reps, key="ms"):
    order = sorted(range(len(reps)), key=lambda i: reps[i][key] if key == "ms" else reps[i][key]["ms"])
    return reps[order[len(order) // 2]]


def measure_h2d(torch, nbytes, reps=12, store=None):
    """Pinned host -> device copy rate (GB/s): the better of a train of expert-sized copies and one large
    copy, best of `reps`, CUDA events on the copying stream.  Sources: a fresh pinned buffer and, when given,
    the head of the expert store itself (`store`: pinned uint8 tensor) -- the memory the steps fetch from,
    which may sit on another NUMA node than a fresh allocation."""
    n_copies = int(min(256, max(32, -(-(512 << 20) // nbytes))))        # at least 512 MB per pass where that takes <= 256 copies
    fresh = torch.empty(n_copies * nbytes, dtype=torch.uint8).pin_memory()
    fresh.fill_(1)
    sources = [fresh]
    if store is not None and store.numel() >= n_copies * nbytes:
        sources.append(store[:n_copies * nbytes])
    d = torch.empty(n_copies * nbytes, dtype=torch.uint8, device="cuda")
    st = torch.cuda.Stream()
    best = 0.0
    with torch.cuda.stream(st):
        for h in sources:
            for rep in range(reps + 2):
                for pieces in (n_copies, 1):
                    chunk = n_copies * nbytes // pieces
                    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    torch.cuda.synchronize()
                    a.record(st)
                    for i in range(pieces):
                        d[i * chunk:(i + 1) * chunk].copy_(h[i * chunk:(i + 1) * chunk], non_blocking=True)
                    b.record(st)
                    torch.cuda.synchronize()
                    if rep >= 2:                                   # the first passes touch the pages
                        best = max(best, n_copies * nbytes / a.elapsed_time(b) / 1e6)
    return best


def measure_copy_peak(torch):
    """This box's device-to-device copy rate (read + write bytes, GB/s), the way the stored peak was taken:
    b.copy_(a) over 1 Gi bf16 elements, best of 10, CUDA events.  Boxes of the pool differ by a few per cent."""
    n = 1 << 30
    a = torch.empty(n, dtype=torch.bfloat16, device="cuda")
    b = torch.empty_like(a)                      # contents do not matter for a copy
    best = 0.0
    for rep in range(12):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        b.copy_(a)
        e1.record()
        torch.cuda.synchronize()
        if rep >= 2:
            best = max(best, 2 * n * 2 / e0.elapsed_time(e1) / 1e6)
    del a, b
    torch.cuda.empty_cache()
    return best


def reduce_over_ranks(dist, maxima: dict, sums: dict, device):
    """Whole-job figures of N independent replicas: times are the maximum over ranks, counts the
    sum.  `dist` is torch.distributed (initialised) or None for a single process."""
    out = dict(maxima)
    out.update(sums)
    if dist is None:
        return out
    import torch
    for keys, op in ((sorted(maxima), dist.ReduceOp.MAX), (sorted(sums), dist.ReduceOp.SUM)):
        if not keys:
            continue
        t = torch.tensor([float(out[k]) for k in keys], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=op)
        for k, v in zip(keys, t.tolist()):
            out[k] = v
    return out


def step_roofline(shape, r, steps, peak_hbm, h2d_peak):
    """bytes one step must move: resident experts + shared + router from HBM, misses over the host link"""
    # a batched stack over an FP8 or 4-bit store keeps bf16 blocks on the device (widened on arrival)
    if shape.weight_dtype in (2, 3) and shape.batch > 1:
        S_dev = synth.expert_block_elems(shape.hidden, shape.inter_routed) * 2
        S_sh = synth.expert_block_elems(shape.hidden, shape.inter_shared) * 2
    else:
        S_dev, S_sh = synth.expert_block_bytes(shape), synth.expert_block_bytes(shape, shared=True)
    router = shape.n_layers * shape.n_routed * shape.hidden * (4 if shape.weight_dtype == 0 else 2)
    hbm = (r["uniq_hits"] + r["uniq_misses"]) * S_dev / steps + shape.n_layers * shape.n_shared * S_sh + router
    t_hbm = hbm / (peak_hbm * 1e9)
    t_h2d = r["h2d_bytes"] / steps / (h2d_peak * 1e9)
    t_roof = max(t_hbm, t_h2d)
    return {"t_hbm_ms": t_hbm * 1e3, "t_h2d_ms": t_h2d * 1e3, "t_step_ms": r["ms"] / steps,
            "frac": t_roof / (r["ms"] / steps / 1e3), "bound": "h2d" if t_h2d > t_hbm else "hbm",
            "h2d_achieved_gbs": r["h2d_bytes"] / (r["ms"] / 1e3) / 1e9}


def summarise(shape, r, steps, peak_hbm, h2d_peak):
    return {"tokens_per_s": steps * shape.batch / (r["ms"] / 1e3), "ms_per_step": r["ms"] / steps,
            "hit_rate": r["uniq_hits"] / max(1, r["uniq_hits"] + r["uniq_misses"]),
            "eor": r["overlap"] / max(1, r["pairs"] * shape.top_k),
            "misses_per_step": r["uniq_misses"] / steps,
            "step_roofline": step_roofline(shape, r, steps, peak_hbm, h2d_peak)}


def all_resident(torch, wl, stream, shape, seed, rho, steps, warmup, peak_hbm, h2d_peak):
    """The same stream on a stack with as many slots as experts (no misses once warm): the expert kernel
    and the whole step against HBM alone."""
    wl_r = copy.copy(wl)
    wl_r.stack = wl.new_stack(shape.n_routed, stream.cuda_stream)
    try:
        r = run_protocol(torch, wl_r, stream, shape, seed, rho, steps, warmup, 1, False, False,
                         prewarm_iid=max(192, 3 * shape.n_routed // max(1, shape.top_k * shape.batch)))[0]
    finally:
        wl_r.stack.close()
    ms_r, n_r, b_r = r["kernel_resident"]
    gbs = b_r / (ms_r / 1e3) / 1e9 if ms_r > 0 else 0.0
    return {"cache_slots": shape.n_routed, "tokens_per_s": steps * shape.batch / (r["ms"] / 1e3),
            "ms_per_step": r["ms"] / steps, "misses": r["uniq_misses"], "kernel_gbs": gbs,
            "kernel_frac_of_measured": gbs / peak_hbm, "kernel_frac_of_nominal_8TBs": gbs / NOMINAL_HBM_GBS,
            "step_frac_of_hbm_roofline": step_roofline(shape, r, steps, peak_hbm, h2d_peak)["frac"]}


def short_run(torch, name, steps, warmup, peak_hbm, h2d_peak_of, store_of=None, max_distinct=8, keep=None):
    """One of the other workloads under the same protocol, one repeat, plus its all-resident run."""
    from paper_2605_27081_b200.loader import LoadedWorkload
    cfg = synth.config(name)
    shape, C, seed = cfg["shape"], cfg["cache_slots"], cfg["seed"]
    S_e = synth.expert_block_bytes(shape)
    distinct = None
    if store_of is None and shape.n_routed > max_distinct and shape.n_layers * shape.n_routed * S_e > 1e9:
        # bound the pinned store and, above all, the time to generate it (seconds per GB on the host cores):
        # expert ids share this many distinct blocks per layer; a fetch moves the same number of bytes from
        # pinned memory whichever block it reads, and routing does not depend on the expert weights
        distinct = max_distinct
    stream = torch.cuda.Stream()
    wl = LoadedWorkload(shape, C, seed, stream=stream.cuda_stream, distinct_experts=distinct, store_of=store_of)
    out = {"kernel": kernel_name(shape), "dtype": DTYPE_NAME[shape.weight_dtype], "batch": shape.batch,
           "cache_slots": C, "steps": steps, "warmup": warmup,
           "distinct_experts_per_layer": wl.n_distinct, "blocks_aliased": wl.n_distinct < shape.n_routed}
    try:
        h2d_peak = h2d_peak_of(S_e, wl._store_t)
        out["h2d_peak_gbs"] = h2d_peak
        runs = {}
        for rho in cfg["rhos"]:
            r = run_protocol(torch, wl, stream, shape, seed, rho, steps, warmup, 1, False, False)[0]
            runs["per_sequence" if rho is None else str(rho)] = summarise(shape, r, steps, peak_hbm, h2d_peak)
        out["runs"] = runs
        rho0 = cfg["rhos"][0]
        out["all_resident"] = all_resident(torch, wl, stream, shape, seed, rho0, min(steps, 64), warmup, peak_hbm,
                                           h2d_peak)
    finally:
        wl.close()
    if keep is not None:
        keep[name] = wl                       # its pinned store may serve a later workload with the same blocks
    return out


def run_ours(args, rank, world, local_rank):
    import torch
    from paper_2605_27081_b200.loader import LoadedWorkload

    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    cfg = synth.config(args.workload)
    shape, C, seed = cfg["shape"], cfg["cache_slots"], cfg["seed"]
    if args.rho is None:
        args.rho = cfg["rhos"][0] if args.workload != "dsv2lite" else 0.9
    if args.layers:
        # a shallower stack of the same layer shape: for profiler captures, not a bench line
        shape = synth.Shape(**{**shape.asdict(), "n_layers": args.layers})
    S_e = synth.expert_block_bytes(shape)
    peak_hbm, peak_kind = measured_peaks()

    # Replicas share the host: keep all pinned stores within the memory that is there.
    avail = os.sysconf("SC_PHYS_PAGES") * os.sysconf("SC_PAGE_SIZE")
    full = shape.n_layers * shape.n_routed * S_e
    distinct = None
    if world * full > 0.6 * avail:
        distinct = max(C + shape.top_k, int(0.6 * avail / world / (shape.n_layers * S_e)))
    if args.distinct:
        distinct = args.distinct
    stream = torch.cuda.Stream()
    wl = LoadedWorkload(shape, C, seed, stream=stream.cuda_stream, distinct_experts=distinct)
    note(f"{args.workload}: store of {wl.n_distinct} distinct blocks per layer loaded")
    h2d_cache = {}

    def h2d_peak_of(nbytes, store=None):
        if nbytes not in h2d_cache:
            h2d_cache[nbytes] = measure_h2d(torch, nbytes, store=store)
        return h2d_cache[nbytes]

    h2d_peak = h2d_peak_of(S_e, wl._store_t)
    copy_here = measure_copy_peak(torch) if rank == 0 else None

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # Headline coefficient: `repeats` repeats of cold start, device-input steps and host-buffer steps.
    barrier()
    reps = run_protocol(torch, wl, stream, shape, seed, args.rho, args.steps, args.warmup, args.repeats, True,
                        not args.no_cold, local_rank=local_rank if rank == 0 else None)
    barrier()
    note("headline repeats done")
    head = median_rep(reps)
    head_e2e = median_rep(reps, "e2e")["e2e"]
    results = {args.rho: head}
    for rho in cfg["rhos"]:
        if rho != args.rho and not args.no_sweep:
            results[rho] = run_protocol(torch, wl, stream, shape, seed, rho, args.steps, args.warmup, 1, False, False)[0]
    barrier()

    resident = None
    if not args.no_resident and rank == 0:
        resident = all_resident(torch, wl, stream, shape, seed, args.rho, min(args.steps, 256), args.warmup, peak_hbm,
                                h2d_peak)

    note("sweep and all-resident done")
    # The same steps through the multi-step entry point (all inputs known up front: step t+1 is routed
    # while step t is still fetching, so the host link stays busy across step boundaries).
    multi = None
    if shape.batch == 1 and not args.no_multi and rank == 0:
        n, w = args.steps, args.warmup
        hid = torch.from_numpy(synth.HiddenStream(seed, shape, args.rho).take(w + n)).to("cuda")
        m_out = torch.empty((n, shape.n_layers, 1, shape.hidden), dtype=torch.float32, device="cuda")
        m_ids = torch.empty((n, shape.n_layers, 1, shape.top_k), dtype=torch.int32, device="cuda")
        m_g = torch.empty((n, shape.n_layers, 1, shape.top_k), dtype=torch.float32, device="cuda")
        wl.stack.cache_reset()
        torch.cuda.synchronize()
        with torch.cuda.stream(stream):
            wl.stack.decode_steps(w, hid[:w], m_out[:w], m_ids[:w], m_g[:w])
            c0 = wl.stack.cache_stats()
            ea, eb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            ea.record(stream)
            wl.stack.decode_steps(n, hid[w:], m_out, m_ids, m_g)
            eb.record(stream)
            torch.cuda.synchronize()
        c1 = wl.stack.cache_stats()
        ms_m = ea.elapsed_time(eb)
        h2d = c1["h2d_bytes"] - c0["h2d_bytes"]
        multi = {"tokens_per_s": n / (ms_m / 1e3), "ms_per_step": ms_m / n, "steps_per_call": n,
                 "misses_per_step": (c1["uniq_misses"] - c0["uniq_misses"]) / n,
                 "h2d_achieved_gbs": h2d / (ms_m / 1e3) / 1e9,
                 "frac_of_h2d_roofline": (h2d / (h2d_peak * 1e9)) / (ms_m / 1e3)}
        del hid, m_out, m_ids, m_g

    # Chained variant (layers joined by a residual): same stack, one route/fetch round trip per layer.
    chained = None
    if shape.batch == 1 and not args.no_chained and rank == 0:
        n = min(args.steps, 128)
        hid = torch.from_numpy(synth.HiddenStream(seed, shape, args.rho).take(args.warmup + n)[:, 0, 0].copy()).to("cuda")
        d_fin = torch.empty(shape.hidden, dtype=torch.float32, device="cuda")
        d_ids = torch.empty((shape.n_layers, 1, shape.top_k), dtype=torch.int32, device="cuda")
        d_g = torch.empty((shape.n_layers, 1, shape.top_k), dtype=torch.float32, device="cuda")
        wl.stack.cache_reset()
        torch.cuda.synchronize()
        with torch.cuda.stream(stream):
            for t in range(args.warmup):
                wl.stack.decode_step_chained(hid[t], d_fin, None, d_ids, d_g)
            c0 = wl.stack.cache_stats()
            ea, eb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            ea.record(stream)
            for t in range(args.warmup, args.warmup + n):
                wl.stack.decode_step_chained(hid[t], d_fin, None, d_ids, d_g)
            eb.record(stream)
            torch.cuda.synchronize()
        c1 = wl.stack.cache_stats()
        ms_c = ea.elapsed_time(eb)
        h2d_c = c1["h2d_bytes"] - c0["h2d_bytes"]
        chained = {"tokens_per_s": n / (ms_c / 1e3), "ms_per_step": ms_c / n,
                   "misses_per_step": (c1["uniq_misses"] - c0["uniq_misses"]) / n,
                   "h2d_achieved_gbs": h2d_c / (ms_c / 1e3) / 1e9,
                   "frac_of_h2d_roofline": (h2d_c / (h2d_peak * 1e9)) / (ms_c / 1e3)}

    red = reduce_over_ranks(dist, {"ms": head["ms"], "e2e_ms": head_e2e["ms"]}, {"launches": head["launches"]}, "cuda")
    ms, e2e_ms, launches = red["ms"], red["e2e_ms"], red["launches"]
    if rank != 0:
        wl.close()
        if dist is not None:
            dist.destroy_process_group()
        return
    tokens = args.steps * world * shape.batch
    value = tokens / (ms / 1e3)

    kname = kernel_name(shape)
    kr_ms, kr_n, kr_b = head["kernel_resident"]
    km_ms, km_n, km_b = head["kernel_miss"]
    ach = kr_b / (kr_ms / 1e3) / 1e9 if kr_ms > 0 else 0.0
    ratio = None if args.layers else TRAFFIC_RATIO.get((args.workload, kname))
    roofline = {"bound": "hbm", "achieved": ach, "peak": peak_hbm, "unit": "GB/s", "frac": ach / peak_hbm,
                "traffic": kr_b / max(1, kr_n) * ratio if ratio else None,
                "peak_kind": f"of {peak_kind}", "kernel": kname + " resident phase",
                "note": "the measured peak is a copy (reads and writes); a read-only stream can run a few per cent above it",
                "launches": kr_n, "avg_launch_ms": kr_ms / max(1, kr_n), "bytes_per_launch": kr_b / max(1, kr_n),
                "frac_of_nominal_8TBs": ach / NOMINAL_HBM_GBS,
                "copy_peak_this_box": copy_here, "frac_of_this_box_copy": ach / copy_here if copy_here else None}
    miss_phase = {"launches": km_n, "avg_launch_us": km_ms * 1e3 / max(1, km_n),
                  "achieved_gbs": km_b / (km_ms / 1e3) / 1e9 if km_ms > 0 else 0.0}

    # CPU baseline: the oracle on a bounded sample, rank 0 only.
    note("multi-step and chained done")
    cpu = None
    if not args.no_cpu_baseline and world == 1:
        cpu = cpu_baseline_legs(shape, C, seed, args.rho, wl.expert_block)
        note("cpu baseline done")

    sweep = {str(rho): summarise(shape, r, args.steps, peak_hbm, h2d_peak) for rho, r in results.items()}
    all_ms = sorted(r["ms"] for r in reps)
    all_e2e = sorted(r["e2e"]["ms"] for r in reps)
    line = {
        "metric": metric_name(shape), "value": value, "unit": "tokens/s",
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": DTYPE_NAME[shape.weight_dtype], "data": "synthetic",
        "config": {"workload": args.workload, "rho": args.rho, "cache_slots": C, "batch": shape.batch,
                   "layers": shape.n_layers,
                   "l2": "inputs larger than L2 (>= 1.6 GB of expert weights streamed per step)",
                   "parallelism": "replicas only" if world > 1 else "single GPU",
                   "distinct_experts_per_layer": wl.n_distinct},
        "repeats": {"n": len(reps), "reported": "median repeat",
                    "tokens_per_s_min_med_max": [args.steps * shape.batch / (m / 1e3) for m in (all_ms[-1], all_ms[len(all_ms) // 2], all_ms[0])],
                    "e2e_tokens_per_s_min_med_max": [args.steps * shape.batch / (m / 1e3) for m in (all_e2e[-1], all_e2e[len(all_e2e) // 2], all_e2e[0])],
                    "note": "every repeat: cold cache, the same warm-up steps, the same timed steps (identical miss sequence)"},
        "clocks": merge_clocks([r.get("clocks") for r in reps]),
        "e2e": {"value": tokens / (e2e_ms / 1e3), "unit": "tokens/s",
                "h2d_bytes_per_step": head_e2e["in_bytes"] + head_e2e["h2d_bytes"] / args.steps,
                "d2h_bytes_per_step": head_e2e["out_bytes"],
                "misses_per_step": head_e2e["uniq_misses"] / args.steps,
                "note": "remoe_decode_step_host on the same steps as `value` (same cold start, warm-up and hidden "
                        "states): hidden states from pinned host memory, outputs read back every step; h2d bytes "
                        "include this leg's own expert fetches"},
        "gpu_launches": int(launches),
        "roofline": roofline,
        "roofline_miss_phase": miss_phase,
        "step_roofline": sweep[str(args.rho)]["step_roofline"],
        "hit_rate": sweep[str(args.rho)]["hit_rate"], "eor": sweep[str(args.rho)]["eor"],
        "h2d_peak_gbs": h2d_peak,
        "sweep": sweep,
        "cpu_baseline": cpu,
    }
    if "cold" in head:
        c = head["cold"]
        line["cold_start"] = dict(summarise(shape, c, c["steps"], peak_hbm, h2d_peak), steps=c["steps"],
                                  note="steps 1..%d from an empty cache (request-isolated start), kernels warm" % c["steps"])
    if resident is not None:
        line["all_resident"] = resident
    if multi is not None:
        line["multi_step"] = multi
    if chained is not None:
        line["chained"] = chained
    wl_keep = wl
    if not args.no_others and world == 1 and not args.layers and args.workload == WORKLOAD:
        others, kept = {}, {}
        n_o, w_o = min(args.steps, 24), min(max(args.warmup, 8), 16)
        for name in ("tiny_fp32", "qwen15moe", "qwen3_30b", "dsv2lite_b32", "dsv2lite_fp8", "dsv2lite_b32_fp8",
                     "dsv2lite_int4", "dsv2lite_b32_int4"):
            if name not in synth.CONFIGS:
                continue
            borrow = None
            if name == "dsv2lite_b32" and wl_keep.n_distinct == shape.n_routed:
                borrow = wl_keep
            if name == "dsv2lite_b32_fp8":
                borrow = kept.get("dsv2lite_fp8")
            if name == "dsv2lite_b32_int4":
                borrow = kept.get("dsv2lite_int4")
            try:
                others[name] = short_run(torch, name, n_o, w_o, peak_hbm, h2d_peak_of, store_of=borrow, keep=kept)
            except Exception as ex:              # a workload that cannot run here must not lose the line
                others[name] = {"error": f"{type(ex).__name__}: {ex}"}
            note(f"other workload {name} done")
        line["other_workloads"] = others
    print(json.dumps(line), flush=True)
    wl.close()
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=256)
    ap.add_argument("--warmup", type=int, default=16)
    ap.add_argument("--repeats", type=int, default=3, help="repeats of the headline protocol (median reported)")
    ap.add_argument("--rho", type=float, default=None, help="AR(1) coefficient of the headline run (default 0.9)")
    ap.add_argument("--workload", default=WORKLOAD, choices=sorted(synth.CONFIGS),
                    help="default: the DeepSeek-V2-Lite-shaped batch-1 stack the metric is quoted on")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--layers", type=int, default=0, help="use only this many layers (profiling captures)")
    ap.add_argument("--distinct", type=int, default=0,
                    help="let expert ids share this many distinct host blocks per layer (quick experiments)")
    ap.add_argument("--no-sweep", action="store_true")
    ap.add_argument("--no-resident", action="store_true")
    ap.add_argument("--no-chained", action="store_true")
    ap.add_argument("--no-multi", action="store_true")
    ap.add_argument("--no-cold", action="store_true")
    ap.add_argument("--no-others", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    args.repeats = max(1, args.repeats)
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        if args.rho is None:
            args.rho = 0.9 if args.workload == "dsv2lite" else synth.config(args.workload)["rhos"][0]
        run_reference(args, rank, world)
    else:
        run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
