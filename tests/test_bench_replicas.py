"""Multi-process aggregation used by bench.py --gpus N (replicas only): two gloo ranks on CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    out = bench.reduce_over_ranks(dist, {"ms": 100.0 + 50.0 * rank, "e2e_ms": 300.0 - 20.0 * rank},
                                  {"launches": 10 + rank}, "cpu")
    dist.barrier()
    q.put((rank, out))
    dist.destroy_process_group()


def test_two_replicas_take_max_time_and_sum_counts():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = dict(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for r in range(2):
        assert got[r] == {"ms": 150.0, "e2e_ms": 300.0, "launches": 21.0}
    # value = tokens of all replicas / slowest replica's time
    steps, world = 64, 2
    assert steps * world / (got[0]["ms"] / 1e3) == 128 / 0.15


def test_single_process_passthrough():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_over_ranks(None, {"ms": 3.0}, {"launches": 7}, "cpu") == {"ms": 3.0, "launches": 7}


def test_step_roofline_and_median_arithmetic():
    """bench.py's bookkeeping on made-up counters: bytes per step, the slower of the two transfer times,
    the fraction against the measured step, the device bytes of an FP8 store under a batched stack, and
    the median repeat."""
    import bench
    import synth

    shape = synth.config("dsv2lite")["shape"]
    S_e = synth.expert_block_bytes(shape)
    assert S_e == 3 * 1408 * 2048 * 2
    steps = 10
    r = {"uniq_hits": 26 * 6 * steps - 280, "uniq_misses": 280, "h2d_bytes": 280 * S_e, "ms": 90.0,
         "overlap": 1000, "pairs": 26 * (steps - 1)}
    rf = bench.step_roofline(shape, r, steps, 6500.0, 55.0)
    hbm = 26 * (64 * 2048 * 2 + 6 * S_e + 2 * S_e)                     # router + K routed + 2 shared blocks per layer
    assert abs(rf["t_hbm_ms"] - hbm / 6500e9 * 1e3) < 1e-9
    assert abs(rf["t_h2d_ms"] - 28 * S_e / 55e9 * 1e3) < 1e-9
    assert rf["bound"] == "h2d" and abs(rf["frac"] - rf["t_h2d_ms"] / 9.0) < 1e-12
    assert abs(rf["h2d_achieved_gbs"] - 280 * S_e / 0.09 / 1e9) < 1e-9
    s = bench.summarise(shape, r, steps, 6500.0, 55.0)
    assert abs(s["tokens_per_s"] - steps / 0.09) < 1e-9 and s["misses_per_step"] == 28.0
    assert abs(s["eor"] - 1000 / (26 * 9 * 6)) < 1e-12
    # FP8 store under a batched stack: fetched bytes are FP8, the bytes streamed from HBM are bf16
    b8 = synth.config("dsv2lite_b32_fp8")["shape"]
    r8 = dict(r, h2d_bytes=280 * synth.expert_block_bytes(b8))
    rf8 = bench.step_roofline(b8, r8, steps, 6500.0, 55.0)
    assert abs(rf8["t_hbm_ms"] - rf["t_hbm_ms"]) < 1e-9 and abs(rf8["t_h2d_ms"] - rf["t_h2d_ms"] / 2) < 1e-9
    # int4: 0.5625 bytes per element on both sides
    i4 = synth.config("dsv2lite_int4")["shape"]
    assert synth.expert_block_bytes(i4) == 3 * 1408 * (1024 + 128)
    reps = [{"ms": 3.0, "e2e": {"ms": 9.0}}, {"ms": 1.0, "e2e": {"ms": 7.0}}, {"ms": 2.0, "e2e": {"ms": 8.0}}]
    assert bench.median_rep(reps)["ms"] == 2.0 and bench.median_rep(reps, "e2e")["e2e"]["ms"] == 8.0
    c = bench.merge_clocks([{"sm_mhz": 1900.0, "sm_max_mhz": 1965.0, "reasons": ["sw_power_cap"], "samples": 3, "power_w_max": 900.0},
                            None, {"sm_mhz": 1965.0, "sm_max_mhz": 1965.0, "reasons": [], "samples": 2, "power_w_max": 500.0}])
    assert c["per_repeat_sm_mhz"] == [1900.0, 1965.0] and c["reasons"] == ["sw_power_cap"] and c["samples"] == 5
    assert bench.metric_name(b8) == "decode tokens/s (batch 32, MoE stack)"
    assert bench.kernel_name(b8) == "ffn_batched_tc_kernel<2048>" and bench.kernel_name(i4) == "ffn_stream_kernel<int4_g32,2048>"
