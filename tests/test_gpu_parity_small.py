"""GPU parity on small shapes: every step of the path against the CPU oracle, element by element."""
import numpy as np
import pytest

import synth

pytestmark = pytest.mark.gpu


def _run(shape, cache_slots, rho, steps, seed=0, dense_steps=2, host_api_every=0, policy=None, beta=0.0):
    import torch
    from paper_2605_27081_b200.loader import LoadedWorkload
    from parity_util import StepChecker, oracle_for

    wl = LoadedWorkload(shape, cache_slots, seed)
    try:
        pol_name = "lru"
        if policy is not None:
            wl.stack.set_policy(policy)
            pol_name = {0: "lru", 1: "fifo", 2: "lfu"}[policy]
        if beta:
            wl.stack.set_reroute_beta(beta)
        chk = StepChecker(wl, oracle_for(wl, pol_name, beta), torch)
        hs = synth.HiddenStream(seed, shape, rho)
        last = None
        for t in range(steps):
            h = hs.step()
            host = bool(host_api_every) and t % host_api_every == host_api_every - 1
            last, _ = chk.step(h, ffn="dense" if t < dense_steps else "selected", host_api=host)
            if t % 4 == 3:
                chk.check_directory()
        chk.check_counters()
        o, p, ir = wl.stack.reuse_stats(-1, want_last_ir=True)
        exp = last["overlap"].reshape(-1)
        assert np.allclose(ir, np.where(exp < 0, -1.0, exp / shape.top_k))
        return chk
    finally:
        wl.close()


def test_tiny_fp32_config_full():
    cfg = synth.config("tiny_fp32")
    chk = _run(cfg["shape"], cfg["cache_slots"], cfg["rhos"][0], cfg["steps"], cfg["seed"], dense_steps=64,
               host_api_every=5)
    assert chk.max_out_err <= 1e-4


@pytest.mark.parametrize("shape,c,rho", [
    (synth.Shape(3, 256, 20, 3, 72, 2, 40, 0, 0, 1, 1), 5, 0.6),        # bf16, shared experts, ragged I
    (synth.Shape(2, 512, 33, 4, 50, 1, 130, 1, 0, 1, 1), 4, 0.8),       # N not a multiple of 32, C = K, sigmoid gate
    (synth.Shape(4, 1024, 128, 8, 24, 0, 0, 0, 1, 1, 1), 32, 0.5),      # renormalised top-8 of 128
    (synth.Shape(2, 2048, 64, 6, 44, 2, 44, 0, 0, 1, 1), 16, 0.9),      # full hidden width
    (synth.Shape(2, 128, 9, 9, 16, 0, 0, 0, 0, 0, 1), 9, 0.3),          # K = N = C, float32
    (synth.Shape(1, 1024, 200, 5, 8, 1, 8, 1, 1, 0, 1), 200, 0.0),      # all resident, float32, N = 200
])
def test_small_shapes(shape, c, rho):
    _run(shape, c, rho, steps=24, seed=1, dense_steps=2, host_api_every=7)


@pytest.mark.parametrize("shape,c,rho", [
    (synth.Shape(2, 256, 256, 32, 8, 0, 0, 0, 1, 1, 1), 40, 0.5),       # largest N and K the kernels take
    (synth.Shape(2, 256, 256, 32, 8, 0, 0, 0, 0, 0, 1), 256, 0.5),      # ... with every expert resident
    (synth.Shape(1, 128, 4, 1, 1, 1, 1, 0, 0, 0, 1), 1, 0.2),           # one channel per expert, K = C = 1
    (synth.Shape(40, 256, 8, 2, 8, 3, 8, 1, 0, 1, 1), 2, 0.9),          # more layers than CTAs get rows
])
def test_extreme_shapes(shape, c, rho):
    _run(shape, c, rho, steps=10, seed=7, dense_steps=1)


@pytest.mark.parametrize("shape,c,rho", [
    (synth.Shape(3, 512, 20, 3, 72, 2, 40, 1, 0, 2, 1), 5, 0.6),        # fp8 expert blocks, bf16 router and gate
    (synth.Shape(2, 2048, 64, 6, 44, 2, 44, 0, 1, 2, 1), 16, 0.9),      # full hidden width
])
def test_fp8_expert_store(shape, c, rho):
    _run(shape, c, rho, steps=16, seed=9, dense_steps=1, host_api_every=5)


@pytest.mark.parametrize("shape,c,rho", [
    (synth.Shape(3, 1024, 20, 3, 72, 2, 40, 1, 0, 3, 1), 5, 0.6),       # int4 grouped blocks, bf16 router and gate
    (synth.Shape(2, 2048, 64, 6, 44, 2, 44, 0, 1, 3, 1), 16, 0.9),      # full hidden width
])
def test_int4_expert_store(shape, c, rho):
    chk = _run(shape, c, rho, steps=16, seed=10, dense_steps=1, host_api_every=5)
    assert chk.max_out_err < 1e-4                # both sides use the exact stored values; fp32 accumulation


def test_int4_store_limits():
    from paper_2605_27081_b200 import binding as B
    rc, _ = B.remoe_stack_create(synth.Shape(2, 512, 16, 2, 32, 0, 0, 0, 0, 3, 1), 4)      # H not 1024 / 2048
    assert rc == B.REMOE_E_UNSUPPORTED
    rc, _ = B.remoe_stack_create(synth.Shape(2, 1024, 16, 2, 40, 0, 0, 0, 0, 3, 4), 4)     # batched needs I % 64 == 0
    assert rc == B.REMOE_E_UNSUPPORTED


def _random_shape(rng, batched):
    """A valid stack shape drawn at random: element type, width, expert count, top-K, capacity, intermediate
    sizes, shared experts, gate, renormalisation."""
    dt = int(rng.choice([1, 2, 3] if batched else [0, 1, 2, 3]))
    widths = {0: [128, 256, 512, 1024], 1: [256, 512, 1024, 2048], 2: [512, 1024, 2048], 3: [1024, 2048]}[dt]
    H = int(rng.choice(widths))
    N = int(rng.integers(2, 41))
    K = int(rng.integers(1, min(N, 8) + 1))
    B = int(rng.integers(2, 25)) if batched else 1
    C = int(rng.integers(K if not batched else 1, N + 1))
    tc_only = batched and dt != 1                        # low-precision batched stacks run on the tensor-core path only
    step = 64 if tc_only or (batched and rng.random() < 0.5) else (8 if batched else 1)
    inter = step * int(rng.integers(1, 3 if step == 64 else (12 if step == 8 else 90)))
    S = int(rng.integers(0, 3))
    Is = step * int(rng.integers(1, 3 if step == 64 else (8 if step == 8 else 60))) if S else 0
    return synth.Shape(int(rng.integers(1, 5)), H, N, K, inter, S, Is, int(rng.integers(0, 2)) if S else 0,
                       int(rng.integers(0, 2)), dt, B), C


@pytest.mark.parametrize("seed", range(16))
def test_random_batch1_shapes(seed):
    rng = np.random.default_rng(1000 + seed)
    shape, c = _random_shape(rng, batched=False)
    policy = int(rng.integers(0, 3))
    beta = float(rng.choice([0.0, 0.0, 0.4]))
    _run(shape, c, float(rng.choice([0.0, 0.5, 0.9])), steps=10, seed=seed, dense_steps=1, host_api_every=4,
         policy=policy, beta=beta)


def test_many_layers_span_ctas():
    """Enough rows that CTAs cross expert and layer boundaries in the streaming kernel."""
    shape = synth.Shape(12, 512, 16, 4, 300, 1, 300, 0, 0, 1, 1)
    _run(shape, 6, 0.7, steps=12, seed=2, dense_steps=1)


def test_long_streams_per_cta():
    """Hundreds of weight rows per CTA: the stage ring wraps many times, so every stage's
    barriers go through many phases (a ring whose stages change hands between warps would
    let a warp run a phase ahead of the data)."""
    shape = synth.Shape(4, 2048, 12, 6, 1280, 2, 640, 0, 0, 1, 1)
    _run(shape, 8, 0.8, steps=10, seed=6, dense_steps=0)


@pytest.mark.parametrize("policy", [1, 2])
def test_other_policies(policy):
    _run(synth.Shape(2, 256, 24, 3, 16, 0, 0, 0, 0, 0, 1), 5, 0.5, steps=60, seed=3, dense_steps=0, policy=policy)


def test_reroute_beta():
    _run(synth.Shape(2, 256, 24, 3, 16, 0, 0, 0, 0, 0, 1), 5, 0.3, steps=40, seed=4, dense_steps=0, beta=0.5)


def test_reset_and_errors():
    import torch
    from paper_2605_27081_b200 import binding as B
    from paper_2605_27081_b200.loader import LoadedWorkload
    from parity_util import StepChecker, oracle_for

    shape = synth.Shape(2, 256, 16, 2, 32, 0, 0, 0, 0, 0, 1)
    rc, h = B.remoe_stack_create(shape, 1)
    assert rc == B.REMOE_E_CAPACITY
    rc, h = B.remoe_stack_create(synth.Shape(2, 250, 16, 2, 32), 4)
    assert rc == B.REMOE_E_UNSUPPORTED
    rc, h = B.remoe_stack_create(synth.Shape(0, 256, 16, 2, 32), 4)
    assert rc == B.REMOE_E_ARG
    rc, h = B.remoe_stack_create(shape, 4)
    assert rc == 0
    x = torch.zeros((2, 1, 256), device="cuda")
    ids = torch.zeros((2, 1, 2), dtype=torch.int32, device="cuda")
    g = torch.zeros((2, 1, 2), device="cuda")
    assert B.remoe_decode_step(h, x, x.clone(), ids, g) == B.REMOE_E_NOT_LOADED
    assert B.remoe_decode_step(h, None, x, ids, g) == B.REMOE_E_ARG
    pageable = np.zeros(3 * 256 * 32, np.float32)
    assert B.remoe_load_experts_host(h, 0, 0, [pageable]) == B.REMOE_E_NOT_PINNED
    assert B.remoe_load_experts_host(h, 0, 15, [pageable, pageable]) == B.REMOE_E_ARG
    assert B.remoe_load_router(h, 5, pageable) == B.REMOE_E_ARG
    B.remoe_stack_destroy(h)

    wl = LoadedWorkload(shape, 4, seed=5)
    try:
        chk = StepChecker(wl, oracle_for(wl), torch)
        hs = synth.HiddenStream(5, shape, 0.5).take(10)
        for t in range(6):
            chk.step(hs[t])
        wl.stack.cache_reset()
        chk.o.reset()
        for t in range(10):
            chk.step(hs[t])
        chk.check_counters()
    finally:
        wl.close()


@pytest.mark.parametrize("shape,c", [
    (synth.Shape(6, 512, 24, 3, 64, 1, 32, 1, 0, 1, 1), 6),
    (synth.Shape(4, 256, 16, 2, 40, 0, 0, 0, 1, 0, 1), 4),
    (synth.Shape(5, 128, 12, 2, 24, 1, 16, 0, 0, 0, 1), 2),        # narrowest width: the link kernel's column slices are 16 wide
    (synth.Shape(4, 2048, 32, 4, 24, 2, 16, 1, 0, 3, 1), 6),       # full width, 4-bit grouped store, sigmoid gate
    (synth.Shape(4, 1024, 32, 4, 24, 0, 0, 0, 0, 2, 1), 4),        # FP8 store, C = K
])
def test_chained_stack(shape, c):
    """Layers feeding each other through the residual: routing of layer l+1 sees layer l's output."""
    import torch
    from paper_2605_27081_b200.loader import LoadedWorkload
    from parity_util import StepChecker, oracle_for

    wl = LoadedWorkload(shape, c, seed=8)
    try:
        chk = StepChecker(wl, oracle_for(wl), torch)
        hs = synth.HiddenStream(8, synth.Shape(**{**shape.asdict(), "n_layers": 1}), 0.8)
        for t in range(12):
            chk.step_chained(hs.step()[0, 0])
        chk.check_counters()
    finally:
        wl.close()


def test_non_finite_input_is_reported_not_faulted():
    """NaN hidden states make the top-K undefined; the kernels' own index checks turn that into the
    device-flag status, the context stays usable and a reset clears the condition."""
    import torch
    from paper_2605_27081_b200 import binding as B
    from paper_2605_27081_b200.loader import LoadedWorkload
    from parity_util import StepChecker, oracle_for

    shape = synth.Shape(2, 256, 64, 6, 16, 0, 0, 0, 0, 1, 1)
    wl = LoadedWorkload(shape, 8, seed=12)
    try:
        x = torch.full((2, 1, 256), float("nan"), device="cuda")
        out = torch.empty_like(x)
        ids = torch.zeros((2, 1, 6), dtype=torch.int32, device="cuda")
        g = torch.zeros((2, 1, 6), device="cuda")
        rc = B.remoe_decode_step(wl.stack.h, x, out, ids, g)
        torch.cuda.synchronize()
        rc2 = B.remoe_decode_step(wl.stack.h, x, out, ids, g)
        assert B.REMOE_E_DEVICE_FLAG in (rc, rc2)
        assert "out of range" in B.remoe_last_cuda_error(wl.stack.h)
        torch.cuda.synchronize()
        wl.stack.cache_reset()
        chk = StepChecker(wl, oracle_for(wl), torch)
        hs = synth.HiddenStream(12, shape, 0.5)
        for _ in range(5):
            chk.step(hs.step())
        chk.check_counters()
    finally:
        wl.close()


@pytest.mark.parametrize("host_api", [False, True])
def test_wait_that_runs_out_is_reported_and_reset_restores_service(monkeypatch, host_api):
    """Failure detection without a fault: a stack created with REMOE_FAULT_INJECT=lost_copy runs its
    first resident-phase expert launch with a short wait limit and never issues the copy of that launch's
    first weight row.  The consumer's bounded wait runs out, the kernel records the error and returns (no
    trap, no hang, the context stays usable).  The step through host buffers reports its own failure;
    the step on device buffers has already returned when the kernel runs, so the next synchronising call
    reports it.  A reset clears the condition and the stack then matches the oracle step for step."""
    import torch
    from paper_2605_27081_b200 import binding as B
    from paper_2605_27081_b200.loader import LoadedWorkload
    from parity_util import StepChecker, oracle_for

    shape = synth.Shape(2, 256, 16, 2, 24, 1, 40, 0, 0, 1, 1)        # a shared expert: step 1 has resident rows
    monkeypatch.setenv("REMOE_FAULT_INJECT", "lost_copy")
    wl = LoadedWorkload(shape, 4, seed=21)
    monkeypatch.delenv("REMOE_FAULT_INJECT")
    try:
        hs = synth.HiddenStream(21, shape, 0.5).take(8)
        x = torch.from_numpy(hs[0]).to("cuda")
        out = torch.empty_like(x)
        ids = torch.zeros((2, 1, 2), dtype=torch.int32, device="cuda")
        g = torch.zeros((2, 1, 2), device="cuda")
        if host_api:
            o_h, i_h, g_h = np.empty((2, 1, 256), np.float32), np.empty((2, 1, 2), np.int32), np.empty((2, 1, 2), np.float32)
            assert B.remoe_decode_step_host(wl.stack.h, hs[0], o_h, i_h, g_h) == B.REMOE_E_DEVICE_FLAG
        else:
            assert B.remoe_decode_step(wl.stack.h, x, out, ids, g) == B.REMOE_OK
            torch.cuda.synchronize()                                  # the kernel has returned by itself
            rc, _ = B.remoe_cache_stats(wl.stack.h, -1)
            assert rc == B.REMOE_E_DEVICE_FLAG
            assert B.remoe_decode_step(wl.stack.h, x, out, ids, g) == B.REMOE_E_DEVICE_FLAG
        assert "bounded wait" in B.remoe_last_cuda_error(wl.stack.h)
        torch.cuda.synchronize()
        wl.stack.cache_reset()
        chk = StepChecker(wl, oracle_for(wl), torch)
        for t in range(8):
            chk.step(hs[t], host_api=(t % 2 == 1))
        chk.check_counters()
    finally:
        wl.close()


def test_schedule_order_checker_on_every_path(monkeypatch):
    """REMOE_CHECK_ORDER=1: the host-side ledger replays every launch, copy, event record and wait of the
    scheduler and checks each slot write against the slot's earlier readers and each read against the
    write that filled it.  Single steps, the multi-step call (routes ahead on a third stream), the chained
    step and both batched schedules (copies straight into slots; copies into the staging pool) run under
    it at cache sizes that evict all the time; a call that enqueued an unordered access would return
    REMOE_E_ORDER (and the binding would raise)."""
    import torch
    from paper_2605_27081_b200.loader import LoadedWorkload

    monkeypatch.setenv("REMOE_CHECK_ORDER", "1")

    def drive(shape, c, steps, mode):
        wl = LoadedWorkload(shape, c, seed=31)
        try:
            L, B, H, K = shape.n_layers, shape.batch, shape.hidden, shape.top_k
            hid = torch.from_numpy(synth.HiddenStream(31, shape, 0.3).take(steps)).to("cuda")
            out = torch.empty((steps, L, B, H), device="cuda")
            ids = torch.empty((steps, L, B, K), dtype=torch.int32, device="cuda")
            g = torch.empty((steps, L, B, K), device="cuda")
            if mode == "multi":
                wl.stack.decode_steps(steps // 2, hid, out, ids, g)
                wl.stack.decode_step(hid[steps // 2], out[0], ids[0], g[0])       # back to the single-step path
                wl.stack.decode_steps(steps - steps // 2 - 1, hid[steps // 2 + 1:], out, ids, g)
            elif mode == "chained":
                fin = torch.empty((B, H), device="cuda")
                for t in range(steps):
                    wl.stack.decode_step_chained(hid[t, 0], fin, None, ids[0], g[0])
            else:
                for t in range(steps):
                    wl.stack.decode_step(hid[t], out[t], ids[t], g[t])
            torch.cuda.synchronize()
            compared, bad = wl.stack.order_check_counts()
            assert bad == 0 and compared > 10 * steps, (mode, compared, bad)
            assert wl.stack.cache_stats()["uniq_misses"] > steps
        finally:
            wl.close()

    b1 = synth.Shape(4, 256, 16, 3, 24, 1, 8, 0, 0, 1, 1)
    drive(b1, 3, 40, "single")                      # C = K: every slot may be replaced at every step
    drive(b1, 4, 41, "multi")
    drive(b1, 3, 20, "chained")
    drive(synth.Shape(3, 256, 16, 2, 40, 1, 24, 0, 0, 1, 6), 5, 20, "single")     # batched, mma.sync kernel: copies into slots
    drive(synth.Shape(3, 512, 24, 3, 64, 1, 64, 0, 0, 1, 12), 8, 20, "single")    # batched, tcgen05 kernel: staging pool
    drive(synth.Shape(3, 512, 24, 3, 64, 1, 64, 0, 0, 2, 12), 8, 12, "single")    # the same over an FP8 store
    drive(synth.Shape(3, 512, 24, 3, 64, 1, 64, 0, 0, 1, 12), 8, 8, "chained")
    monkeypatch.delenv("REMOE_CHECK_ORDER")
    wl = LoadedWorkload(b1, 3, seed=31)
    try:
        assert wl.stack.order_check_counts() == (0, 0)              # off unless asked for
    finally:
        wl.close()


def test_policy_switch_and_second_stack_share_a_store():
    """Two stacks over the same pinned store (different capacity and policy) stay independent."""
    import torch
    from paper_2605_27081_b200.loader import LoadedWorkload
    from parity_util import StepChecker, oracle_for
    import copy

    shape = synth.Shape(2, 256, 16, 2, 24, 1, 8, 0, 0, 1, 1)
    wl = LoadedWorkload(shape, 4, seed=13)
    wl2 = copy.copy(wl)
    wl2.cache_slots = 7
    wl2.stack = wl.new_stack(7)
    try:
        wl2.stack.set_policy(1)
        a = StepChecker(wl, oracle_for(wl), torch)
        b = StepChecker(wl2, oracle_for(wl2, "fifo"), torch)
        hs = synth.HiddenStream(13, shape, 0.6)
        for _ in range(25):
            h = hs.step()
            a.step(h)
            b.step(h)
        a.check_counters()
        b.check_counters()
        assert a.o.uniq_misses != b.o.uniq_misses
    finally:
        wl2.stack.close()
        wl.close()


@pytest.mark.parametrize("shape,c,rho,n", [
    (synth.Shape(6, 512, 24, 3, 64, 1, 32, 1, 0, 1, 1), 6, 0.6, 23),       # odd number of steps, sigmoid gate
    (synth.Shape(3, 1024, 40, 4, 200, 2, 100, 0, 1, 1, 1), 9, 0.3, 16),    # many misses per step, renormalised
    (synth.Shape(2, 256, 16, 2, 32, 0, 0, 0, 0, 0, 1), 2, 0.0, 9),         # float32, C = K: every slot turns over
    (synth.Shape(3, 1024, 24, 3, 72, 1, 40, 0, 0, 2, 1), 4, 0.4, 12),      # FP8 store
    (synth.Shape(3, 1024, 24, 3, 72, 1, 40, 0, 0, 3, 1), 4, 0.4, 12),      # 4-bit grouped store
])
def test_multi_step_call_equals_single_steps(shape, c, rho, n):
    """remoe_decode_steps routes step t+1 while step t is still fetching; everything it returns must be
    bit-identical to n calls of remoe_decode_step (itself checked against the oracle above), including
    when single and multi-step calls are mixed on one stack."""
    import torch
    from paper_2605_27081_b200.loader import LoadedWorkload

    wl = LoadedWorkload(shape, c, seed=11)
    other = wl.new_stack(c)
    try:
        L, H, K = shape.n_layers, shape.hidden, shape.top_k
        hid = torch.from_numpy(synth.HiddenStream(11, shape, rho).take(n + 4)).to("cuda")
        out1 = torch.empty((n + 4, L, 1, H), device="cuda")
        ids1 = torch.empty((n + 4, L, 1, K), dtype=torch.int32, device="cuda")
        g1 = torch.empty((n + 4, L, 1, K), device="cuda")
        out2, ids2, g2 = torch.empty_like(out1), torch.empty_like(ids1), torch.empty_like(g1)
        for t in range(n + 4):
            wl.stack.decode_step(hid[t], out1[t], ids1[t], g1[t])
        # 2 single steps, n in one call, 1 single step, 1 in a call of its own
        for t in range(2):
            other.decode_step(hid[t], out2[t], ids2[t], g2[t])
        other.decode_steps(n, hid[2:], out2[2:], ids2[2:], g2[2:])
        other.decode_step(hid[n + 2], out2[n + 2], ids2[n + 2], g2[n + 2])
        other.decode_steps(1, hid[n + 3:], out2[n + 3:], ids2[n + 3:], g2[n + 3:])
        torch.cuda.synchronize()
        assert torch.equal(ids1, ids2) and torch.equal(g1, g2)
        assert torch.equal(out1, out2)
        a, b = wl.stack.cache_stats(), other.cache_stats()
        assert a == b and a["uniq_misses"] > 0
        assert wl.stack.reuse_stats() == other.reuse_stats()
        ta, tb = wl.stack.last_step_trace(), other.last_step_trace()
        for k in ta:
            assert np.array_equal(ta[k], tb[k]), k
        ua, ha = wl.stack.step_history()
        ub, hb = other.step_history()
        assert list(ua) == list(ub) and list(ha) == list(hb)
        ca, cb = wl.stack.expert_load()[0], other.expert_load()[0]
        assert np.array_equal(ca, cb)
    finally:
        other.close()
        wl.close()
