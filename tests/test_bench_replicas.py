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
