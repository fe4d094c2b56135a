#!/usr/bin/env python
"""Decode-throughput benchmark of the bounded-cache MoE decode step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--rho R] [--impl ours|reference]

A "step" is one decode step: one token through all MoE layers of the DeepSeek-V2-Lite-shaped
stack (26 layers, hidden 2048, 64 routed experts top-6 + 2 shared, intermediate 1408, bf16
weights, 16 cache slots per layer, LRU), driven by seeded AR(1) hidden states.  One JSON line
is printed by rank 0.  With N > 1 every rank runs an independent replica (the path has no
exchange step); the time is the maximum over ranks and the value the sum of tokens.
"""
from __future__ import annotations

import argparse
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
# DRAM bytes (read + write) per algorithmic byte of a resident-phase launch, from the ncu capture
# summarised in profiles/ffn_stream_{bf16,fp8}_h2048_4layers_ncu_full.md (traffic grows in proportion to the
# blocks streamed); only valid for the kernel and shape it was taken on.
TRAFFIC_RATIO = {("dsv2lite", 1): 1.009, ("dsv2lite_fp8", 2): 1.018, ("dsv2lite_b32", 1): None}
DTYPE_NAME = {0: "f32", 1: "bf16", 2: "fp8_e4m3"}      # weight storage; accumulation is always f32
CLOCK_QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
               "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
               "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")


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
                                       "--format=csv,noheader,nounits", "-lms", "200"],
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


def oracle_sample(shape, cache_slots, seed, rho, layers, steps, warmup=0):
    """Time the CPU oracle (as it stands) on `layers` layers for `steps` decode steps."""
    from oracle import remoe_oracle as orc
    sub = synth.Shape(**{**shape.asdict(), "n_layers": layers})

    def widen(a):
        return synth.bf16_bits_to_f32(a) if shape.weight_dtype == 1 else a

    routers = [widen(synth.gen_router(seed, shape, l)) for l in range(layers)]
    blocks = {}

    def ew(l, e):
        if (l, e) not in blocks:
            blocks[(l, e)] = widen(synth.gen_expert_block(seed, shape, l, e))
        return synth.expert_matrices(blocks[(l, e)], shape.hidden, shape.inter_routed)

    shared = {(l, i): widen(synth.gen_shared_block(seed, shape, l, i)) for l in range(layers)
              for i in range(shape.n_shared)}

    def sw(l, i):
        return synth.expert_matrices(shared[(l, i)], shape.hidden, shape.inter_shared)

    st = orc.OracleStack(sub, cache_slots, routers, ew, sw)
    hs = synth.HiddenStream(seed, shape, rho)
    hidden = [hs.step()[:layers] for _ in range(warmup + steps)]
    # weights are generated before the clock starts (the GPU side also starts with its store ready)
    for t in range(warmup + steps):
        r = st.step(hidden[t], ffn=None)
        for l in range(layers):
            for e in r["ids"][l].reshape(-1):
                ew(l, int(e))
    st.reset()
    for t in range(warmup):
        st.step(hidden[t], ffn="selected")
    t0 = time.perf_counter()
    for t in range(warmup, warmup + steps):
        st.step(hidden[t], ffn="selected")
    dt = time.perf_counter() - t0
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        cores = 1
    return dt, cores


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
    sample = (f"{args.steps} decode steps over the first {layers} of {shape.n_layers} layers, time scaled by "
              f"{shape.n_layers}/{layers}; selected-experts-only fp64 oracle")
    line = {
        "impl": "reference", "metric": "decode tokens/s (batch 1, MoE stack)", "value": value, "unit": "tokens/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": per_step * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "rho": args.rho, "cache_slots": cfg["cache_slots"], "batch": shape.batch},
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def timed_steps(torch, wl, stream, d_hidden, d_out, d_ids, d_g, first, count):
    """Run `count` decode steps from device-resident inputs; returns elapsed ms (CUDA events)."""
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    with torch.cuda.stream(stream):
        a.record(stream)
        for t in range(first, first + count):
            wl.stack.decode_step(d_hidden[t], d_out, d_ids, d_g)
        b.record(stream)
    torch.cuda.synchronize()
    return a.elapsed_time(b)


def run_rho(torch, wl, stream, shape, seed, rho, steps, warmup, with_e2e, prewarm_iid=0):
    """Cold cache -> warm-up -> K timed steps (device inputs) [-> K timed steps through host buffers]."""
    L, H, K, B = shape.n_layers, shape.hidden, shape.top_k, shape.batch
    n = warmup + steps * (2 if with_e2e else 1)
    hidden = synth.HiddenStream(seed, shape, rho).take(n)
    h_pinned = torch.from_numpy(hidden).pin_memory()
    d_hidden = h_pinned.to("cuda", non_blocking=False)
    d_out = torch.empty((L, B, H), dtype=torch.float32, device="cuda")
    d_ids = torch.empty((L, B, K), dtype=torch.int32, device="cuda")
    d_g = torch.empty((L, B, K), dtype=torch.float32, device="cuda")
    st = wl.stack
    st.cache_reset()
    st.set_profiling(False)
    torch.cuda.synchronize()
    if prewarm_iid:
        # independent hidden states touch every expert quickly, so a cache as large as the expert
        # set ends up holding all of them before the measured stream starts
        d_pre = torch.from_numpy(synth.HiddenStream(seed + 1, shape, 0.0).take(prewarm_iid)).to("cuda")
        timed_steps(torch, wl, stream, d_pre, d_out, d_ids, d_g, 0, prewarm_iid)
    timed_steps(torch, wl, stream, d_hidden, d_out, d_ids, d_g, 0, warmup)
    c0, l0 = st.cache_stats(), st.launch_count()
    ov0 = st.reuse_stats()
    st.set_profiling(True)
    ms = timed_steps(torch, wl, stream, d_hidden, d_out, d_ids, d_g, warmup, steps)
    c1, l1 = st.cache_stats(), st.launch_count()
    ov1 = st.reuse_stats()
    k_res = st.kernel_time(0)
    k_miss = st.kernel_time(1)
    st.set_profiling(False)
    res = {
        "ms": ms, "launches": l1 - l0,
        "uniq_hits": c1["uniq_hits"] - c0["uniq_hits"], "uniq_misses": c1["uniq_misses"] - c0["uniq_misses"],
        "h2d_bytes": c1["h2d_bytes"] - c0["h2d_bytes"],
        "overlap": ov1[0] - ov0[0], "pairs": ov1[1] - ov0[1],
        "kernel_resident": k_res, "kernel_miss": k_miss,
    }
    if with_e2e:
        out_h = torch.empty((L, B, H), dtype=torch.float32).pin_memory().numpy()
        ids_h = torch.empty((L, B, K), dtype=torch.int32).pin_memory().numpy()
        g_h = torch.empty((L, B, K), dtype=torch.float32).pin_memory().numpy()
        hp = h_pinned.numpy()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        a.record(stream)
        for t in range(warmup + steps, warmup + 2 * steps):
            st.decode_step_host(hp[t], out_h, ids_h, g_h)
        b.record(stream)
        torch.cuda.synchronize()
        wall = (time.perf_counter() - t0) * 1e3
        res["e2e_ms"] = max(a.elapsed_time(b), wall)
        res["e2e_in_bytes"] = hp[0].nbytes
        res["e2e_out_bytes"] = out_h.nbytes + ids_h.nbytes + g_h.nbytes
    return res


def measure_h2d(torch, nbytes, reps=12):
    """Pinned host -> device copy rate (GB/s): the better of a train of expert-sized copies and
    one large copy, best of `reps`, CUDA events on the copying stream."""
    n_copies = 32
    h = torch.empty(n_copies * nbytes, dtype=torch.uint8).pin_memory()
    h.fill_(1)
    d = torch.empty(n_copies * nbytes, dtype=torch.uint8, device="cuda")
    st = torch.cuda.Stream()
    best = 0.0
    with torch.cuda.stream(st):
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
                if rep >= 2:                                   # the first rounds touch the pages
                    best = max(best, n_copies * nbytes / a.elapsed_time(b) / 1e6)
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
    stream = torch.cuda.Stream()
    wl = LoadedWorkload(shape, C, seed, stream=stream.cuda_stream, distinct_experts=distinct)
    h2d_peak = measure_h2d(torch, S_e)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    rhos = [args.rho] + [r for r in cfg["rhos"] if r != args.rho and not args.no_sweep]
    results = {}
    clocks = None
    for rho in rhos:
        is_head = rho == args.rho
        barrier()
        sampler = ClockSampler(local_rank) if (is_head and rank == 0) else None
        results[rho] = run_rho(torch, wl, stream, shape, seed, rho, args.steps, args.warmup, with_e2e=is_head)
        barrier()
        if sampler is not None:
            clocks = sampler.stop()

    # All-resident stack (C = N, no misses once warm): the expert-streaming kernel against HBM.
    resident = None
    if not args.no_resident and rank == 0:
        import copy
        wl_r = copy.copy(wl)
        wl_r.stack = wl.new_stack(shape.n_routed, stream.cuda_stream)
        r = run_rho(torch, wl_r, stream, shape, seed, args.rho, min(args.steps, 256), args.warmup, False,
                    prewarm_iid=192)
        resident = r
        wl_r.stack.close()

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
        chained = {"tokens_per_s": n / (ms_c / 1e3), "ms_per_step": ms_c / n,
                   "misses_per_step": (c1["uniq_misses"] - c0["uniq_misses"]) / n,
                   "h2d_achieved_gbs": (c1["h2d_bytes"] - c0["h2d_bytes"]) / (ms_c / 1e3) / 1e9}

    head = results[args.rho]
    red = reduce_over_ranks(dist, {"ms": head["ms"], "e2e_ms": head["e2e_ms"]}, {"launches": head["launches"]},
                            "cuda")
    ms, e2e_ms, launches = red["ms"], red["e2e_ms"], red["launches"]
    if rank != 0:
        wl.close()
        if dist is not None:
            dist.destroy_process_group()
        return
    tokens = args.steps * world * shape.batch
    value = tokens / (ms / 1e3)
    per_step_ms = ms / args.steps

    def step_roofline(r, steps):
        # bytes one step must move: resident experts + shared + router from HBM, misses over the host link
        router = shape.n_layers * shape.n_routed * shape.hidden * shape.elem_bytes
        hbm = (r["uniq_hits"] + r["uniq_misses"]) * S_e / steps + shape.n_layers * shape.n_shared * \
            synth.expert_block_bytes(shape, shared=True) + router
        t_hbm = hbm / (peak_hbm * 1e9)
        t_h2d = r["h2d_bytes"] / steps / (h2d_peak * 1e9)
        t_roof = max(t_hbm, t_h2d)
        return {"t_hbm_ms": t_hbm * 1e3, "t_h2d_ms": t_h2d * 1e3, "t_step_ms": r["ms"] / steps,
                "frac": t_roof / (r["ms"] / steps / 1e3), "bound": "h2d" if t_h2d > t_hbm else "hbm",
                "h2d_achieved_gbs": r["h2d_bytes"] / (r["ms"] / 1e3) / 1e9}

    kr_ms, kr_n, kr_b = head["kernel_resident"]
    km_ms, km_n, km_b = head["kernel_miss"]
    ach = kr_b / (kr_ms / 1e3) / 1e9 if kr_ms > 0 else 0.0
    roofline = {"bound": "hbm", "achieved": ach, "peak": peak_hbm, "unit": "GB/s", "frac": ach / peak_hbm,
                "traffic": (kr_b / max(1, kr_n) * TRAFFIC_RATIO[(args.workload, shape.weight_dtype)]
                            if TRAFFIC_RATIO.get((args.workload, shape.weight_dtype)) and not args.layers else None),
                "peak_kind": f"of {peak_kind}", "kernel": kernel_name(shape) + " resident phase",
                "launches": kr_n, "avg_launch_ms": kr_ms / max(1, kr_n), "bytes_per_launch": kr_b / max(1, kr_n),
                "frac_of_nominal_8TBs": ach / NOMINAL_HBM_GBS}
    miss_phase = {"launches": km_n, "avg_launch_us": km_ms * 1e3 / max(1, km_n),
                  "achieved_gbs": km_b / (km_ms / 1e3) / 1e9 if km_ms > 0 else 0.0}

    # CPU baseline: the oracle on a bounded sample, rank 0 only.
    cpu = None
    if not args.no_cpu_baseline and world == 1:
        layers, steps_cpu = 2, 3
        dt, cores = oracle_sample(shape, C, seed, args.rho, layers, steps_cpu)
        per = dt / steps_cpu * shape.n_layers / layers
        cpu = {"value": shape.batch / per, "unit": "tokens/s", "cores": cores, "kind": "oracle",
               "sample": f"first {steps_cpu} decode steps (cold cache) over the first {layers} of {shape.n_layers} "
                         f"layers, time scaled by {shape.n_layers}/{layers}; selected-experts-only fp64 oracle"}

    sweep = {}
    for rho, r in results.items():
        sweep[str(rho)] = {
            "tokens_per_s": args.steps * shape.batch / (r["ms"] / 1e3),
            "hit_rate": r["uniq_hits"] / max(1, r["uniq_hits"] + r["uniq_misses"]),
            "eor": r["overlap"] / max(1, r["pairs"] * shape.top_k),
            "misses_per_step": r["uniq_misses"] / args.steps,
            "step_roofline": step_roofline(r, args.steps)}
    line = {
        "metric": "decode tokens/s (batch 1, MoE stack)", "value": value, "unit": "tokens/s",
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": per_step_ms,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": DTYPE_NAME[shape.weight_dtype], "data": "synthetic",
        "config": {"workload": args.workload, "rho": args.rho, "cache_slots": C, "batch": shape.batch,
                   "layers": shape.n_layers,
                   "l2": "inputs larger than L2 (>= 1.6 GB of expert weights streamed per step)",
                   "parallelism": "replicas only" if world > 1 else "single GPU",
                   "distinct_experts_per_layer": wl.n_distinct},
        "clocks": clocks,
        "e2e": {"value": tokens / (e2e_ms / 1e3), "unit": "tokens/s",
                "h2d_bytes_per_step": head["e2e_in_bytes"] + head["h2d_bytes"] / args.steps,
                "d2h_bytes_per_step": head["e2e_out_bytes"],
                "note": "remoe_decode_step_host: hidden states from pinned host memory, outputs read back; "
                        "h2d bytes include the expert fetches"},
        "gpu_launches": int(launches),
        "roofline": roofline,
        "roofline_miss_phase": miss_phase,
        "step_roofline": sweep[str(args.rho)]["step_roofline"],
        "hit_rate": sweep[str(args.rho)]["hit_rate"], "eor": sweep[str(args.rho)]["eor"],
        "h2d_peak_gbs": h2d_peak,
        "sweep": sweep,
        "cpu_baseline": cpu,
    }
    if resident is not None:
        n = min(args.steps, 256)
        ms_r, n_r, b_r = resident["kernel_resident"]
        line["all_resident"] = {
            "cache_slots": shape.n_routed, "tokens_per_s": n * shape.batch / (resident["ms"] / 1e3),
            "ms_per_step": resident["ms"] / n, "misses": resident["uniq_misses"],
            "kernel_gbs": b_r / (ms_r / 1e3) / 1e9 if ms_r > 0 else 0.0,
            "kernel_frac_of_measured": (b_r / (ms_r / 1e3) / 1e9 / peak_hbm) if ms_r > 0 else 0.0,
            "step_frac_of_hbm_roofline": step_roofline(resident, n)["frac"]}
    if multi is not None:
        line["multi_step"] = multi
    if chained is not None:
        line["chained"] = chained
    print(json.dumps(line), flush=True)
    wl.close()
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=256)
    ap.add_argument("--warmup", type=int, default=16)
    ap.add_argument("--rho", type=float, default=None, help="AR(1) coefficient of the headline run (default 0.9)")
    ap.add_argument("--workload", default=WORKLOAD, choices=sorted(synth.CONFIGS),
                    help="default: the DeepSeek-V2-Lite-shaped batch-1 stack the metric is quoted on")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--layers", type=int, default=0, help="use only this many layers (profiling captures)")
    ap.add_argument("--no-sweep", action="store_true")
    ap.add_argument("--no-resident", action="store_true")
    ap.add_argument("--no-chained", action="store_true")
    ap.add_argument("--no-multi", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
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
