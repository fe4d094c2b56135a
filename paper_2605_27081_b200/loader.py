"""Put a seeded synthetic workload where the library expects it.

Routed experts go to page-locked host memory (the library fetches misses from there),
router and shared-expert weights are copied to the device once.  No arithmetic of the
decode path happens here.
"""
from __future__ import annotations

import numpy as np
import torch

import synth
from .binding import Stack


class LoadedWorkload:
    """A stack plus the host-side tensors it borrows.

    ``distinct_experts``: generate only that many distinct routed blocks per layer and let
    the remaining expert ids alias them (saves host memory and generation time when only
    timing matters); ``None`` generates all N blocks per layer.  ``store_of``: borrow the pinned
    expert store of another loaded workload whose expert blocks are the same tensors (same seed,
    layers, hidden, intermediate size and element type; e.g. the batched variant of a stack) instead
    of generating it again; that workload must outlive this one.
    """

    def __init__(self, shape: synth.Shape, cache_slots: int, seed: int = 0, stream: int | None = None,
                 distinct_experts: int | None = None, threads: int | None = None,
                 store_of: "LoadedWorkload | None" = None):
        self.shape, self.cache_slots, self.seed = shape, cache_slots, seed
        L, N = shape.n_layers, shape.n_routed
        np_dt = {0: np.float32, 1: np.uint16, 2: np.uint8, 3: np.uint8}[shape.weight_dtype]
        blk_bytes = synth.expert_block_bytes(shape)
        elems = blk_bytes // np.dtype(np_dt).itemsize          # stored items per block
        if store_of is not None:
            o = store_of.shape
            same = (o.n_layers, o.hidden, o.inter_routed, o.weight_dtype, o.n_routed, store_of.seed) == \
                   (L, shape.hidden, shape.inter_routed, shape.weight_dtype, N, seed)
            if not same:
                raise ValueError("store_of: the two workloads do not have the same expert blocks")
            nd = store_of.n_distinct
            self.n_distinct = nd
            self._store_t, self.store = store_of._store_t, store_of.store
        else:
            nd = N if distinct_experts is None else min(N, int(distinct_experts))
            self.n_distinct = nd
            gen_shape = synth.Shape(**{**shape.asdict(), "n_routed": nd})
            self._store_t = torch.empty(L * nd * blk_bytes, dtype=torch.uint8, pin_memory=True)
            self.store = self._store_t.numpy().view(np_dt).reshape(L, nd, elems)
            synth.fill_expert_store(seed, gen_shape, self.store, threads=threads)
        self.routers = [synth.gen_router(seed, shape, l) for l in range(L)]
        self.shared_gates = [synth.gen_shared_gate(seed, shape, l) for l in range(L)] if shape.shared_gate else None
        jobs = [(l, i) for l in range(L) for i in range(shape.n_shared)]
        if len(jobs) >= 4:
            from concurrent.futures import ThreadPoolExecutor
            import os
            with ThreadPoolExecutor(threads or len(os.sched_getaffinity(0))) as ex:
                blocks = list(ex.map(lambda li: synth.gen_shared_block(seed, shape, li[0], li[1]), jobs))
        else:
            blocks = [synth.gen_shared_block(seed, shape, l, i) for l, i in jobs]
        self.shared = [[blocks[l * shape.n_shared + i] for i in range(shape.n_shared)] for l in range(L)]

        self.stack = self.new_stack(cache_slots, stream)

    def new_stack(self, cache_slots: int, stream: int | None = None) -> Stack:
        """Another stack (e.g. with a different capacity) borrowing the same host tensors."""
        shape, nd = self.shape, self.n_distinct
        stack = Stack(shape, cache_slots, stream)
        base = self._store_t.data_ptr()
        blk = synth.expert_block_bytes(shape)
        for l in range(shape.n_layers):
            stack.load_router(l, self.routers[l], None if self.shared_gates is None else self.shared_gates[l])
            for i in range(shape.n_shared):
                stack.load_shared(l, i, self.shared[l][i])
            ptrs = [base + (l * nd + (e % nd)) * blk for e in range(shape.n_routed)]
            stack.load_experts_host(l, 0, ptrs, keep=self._store_t)
        return stack

    def expert_block(self, layer: int, expert: int) -> np.ndarray:
        return self.store[layer, expert % self.n_distinct]

    def close(self):
        self.stack.close()
