"""ctypes binding of libremoe.so: argument marshalling only, same names as the C ABI.

Every step of the decode path runs inside the library's CUDA kernels; nothing here
computes.  PyTorch is used by callers for device memory and streams; this module only
needs raw pointers (``tensor.data_ptr()``) and, for host arrays, numpy buffers.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libremoe.so")

REMOE_OK = 0
REMOE_E_ARG, REMOE_E_CAPACITY, REMOE_E_NOT_LOADED, REMOE_E_NOT_PINNED = -1, -2, -3, -4
REMOE_E_CUDA, REMOE_E_DEVICE_FLAG, REMOE_E_UNSUPPORTED, REMOE_E_NOMEM, REMOE_E_ORDER = -5, -6, -7, -8, -9
REMOE_F32, REMOE_BF16, REMOE_FP8_E4M3, REMOE_INT4_G32 = 0, 1, 2, 3
REMOE_POLICY_LRU, REMOE_POLICY_FIFO, REMOE_POLICY_LFU = 0, 1, 2

EXPORTS = [
    "remoe_stack_create", "remoe_load_router", "remoe_load_shared", "remoe_load_experts_host",
    "remoe_decode_step", "remoe_decode_step_host", "remoe_last_step_trace", "remoe_cache_stats",
    "remoe_reuse_stats", "remoe_cache_reset", "remoe_set_policy", "remoe_set_reroute_beta",
    "remoe_set_profiling", "remoe_kernel_time", "remoe_launch_count", "remoe_last_cuda_error", "remoe_stack_destroy",
    "remoe_strerror", "remoe_expert_ffn_static", "remoe_reuse_mass", "remoe_step_history", "remoe_tpot_proxy", "remoe_decode_step_chained",
    "remoe_expert_load", "remoe_decode_steps", "remoe_order_check_counts", "remoe_cache_snapshot",
]


class remoe_shape(C.Structure):
    _fields_ = [(n, C.c_int32) for n in (
        "n_layers", "hidden", "n_routed", "top_k", "inter_routed", "n_shared", "inter_shared",
        "shared_gate", "renorm_topk", "weight_dtype", "batch")]


class remoe_cache_counters(C.Structure):
    _fields_ = [(n, C.c_uint64) for n in (
        "tok_hits", "tok_misses", "uniq_hits", "uniq_misses", "h2d_bytes", "steps")]


class RemoeError(RuntimeError):
    def __init__(self, code, what, detail=""):
        self.code = code
        super().__init__(f"{what}: {code} ({strerror(code)}){' -- ' + detail if detail else ''}")


_lib = None


def lib():
    """The loaded shared library.  There is no fallback: a missing build is an error."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2605_27081_b200.build` "
                "(there is no CPU or PyTorch fallback for this path)")
        L = C.CDLL(LIB_PATH)
        vp, i32, f32p, i32p = C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p
        L.remoe_stack_create.argtypes = [C.POINTER(remoe_shape), i32, vp, C.POINTER(vp)]
        L.remoe_load_router.argtypes = [vp, i32, vp, vp]
        L.remoe_load_shared.argtypes = [vp, i32, i32, vp]
        L.remoe_load_experts_host.argtypes = [vp, i32, i32, i32, C.POINTER(vp)]
        L.remoe_decode_step.argtypes = [vp, f32p, f32p, i32p, f32p]
        L.remoe_decode_step_host.argtypes = [vp, f32p, f32p, i32p, f32p]
        L.remoe_decode_step_chained.argtypes = [vp, f32p, f32p, f32p, i32p, f32p]
        L.remoe_decode_steps.argtypes = [vp, i32, f32p, f32p, i32p, f32p]
        L.remoe_last_step_trace.argtypes = [vp, i32p, i32p, i32p, i32p, i32p]
        L.remoe_cache_stats.argtypes = [vp, i32, C.POINTER(remoe_cache_counters)]
        L.remoe_reuse_stats.argtypes = [vp, i32, C.POINTER(C.c_uint64), C.POINTER(C.c_uint64), vp]
        L.remoe_cache_reset.argtypes = [vp]
        L.remoe_set_policy.argtypes = [vp, i32]
        L.remoe_set_reroute_beta.argtypes = [vp, C.c_float]
        L.remoe_set_profiling.argtypes = [vp, i32]
        L.remoe_kernel_time.argtypes = [vp, i32, C.POINTER(C.c_double), C.POINTER(C.c_uint64), C.POINTER(C.c_uint64)]
        L.remoe_launch_count.argtypes = [vp, C.POINTER(C.c_uint64)]
        L.remoe_cache_snapshot.argtypes = [vp, i32, vp, vp, vp]
        L.remoe_order_check_counts.argtypes = [vp, C.POINTER(C.c_uint64), C.POINTER(C.c_uint64)]
        L.remoe_expert_ffn_static.argtypes = [i32, i32, i32, C.POINTER(vp), C.POINTER(i32), C.POINTER(C.c_float),
                                              vp, vp, vp]
        L.remoe_reuse_mass.argtypes = [vp, i32, C.POINTER(C.c_double), C.POINTER(C.c_uint64), vp]
        L.remoe_step_history.argtypes = [vp, i32, i32, vp, vp, C.POINTER(i32)]
        L.remoe_expert_load.argtypes = [vp, i32, vp, C.POINTER(C.c_double), C.POINTER(C.c_double), C.POINTER(i32)]
        L.remoe_tpot_proxy.argtypes = [vp, i32, C.c_uint64, C.c_double, i32, C.c_double, vp, vp]
        L.remoe_last_cuda_error.argtypes = [vp]
        L.remoe_last_cuda_error.restype = C.c_char_p
        L.remoe_stack_destroy.argtypes = [vp]
        L.remoe_stack_destroy.restype = None
        L.remoe_strerror.argtypes = [C.c_int]
        L.remoe_strerror.restype = C.c_char_p
        for name in EXPORTS:
            if name not in ("remoe_last_cuda_error", "remoe_stack_destroy", "remoe_strerror"):
                getattr(L, name).restype = C.c_int
        _lib = L
    return _lib


def strerror(code: int) -> str:
    return lib().remoe_strerror(int(code)).decode()


def _ptr(x):
    """Raw address of a torch tensor, numpy array, int or None."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    if isinstance(x, np.ndarray):
        return x.ctypes.data
    raise TypeError(type(x))


def _shape_struct(shape) -> remoe_shape:
    if isinstance(shape, remoe_shape):
        return shape
    get = (lambda k: shape[k]) if isinstance(shape, dict) else (lambda k: getattr(shape, k))
    return remoe_shape(*[int(get(n)) for n, _ in remoe_shape._fields_])


# ---- thin wrappers with the C names; each returns the status code (and outputs) ----------

def remoe_stack_create(shape, cache_slots_per_layer: int, cuda_stream: int | None = None):
    h = C.c_void_p()
    st = _shape_struct(shape)
    rc = lib().remoe_stack_create(C.byref(st), int(cache_slots_per_layer), cuda_stream, C.byref(h))
    return rc, h


def remoe_load_router(h, layer, w_router_host, w_shared_gate_host=None):
    return lib().remoe_load_router(h, int(layer), _ptr(w_router_host), _ptr(w_shared_gate_host))


def remoe_load_shared(h, layer, idx, block_host):
    return lib().remoe_load_shared(h, int(layer), int(idx), _ptr(block_host))


def remoe_load_experts_host(h, layer, first_expert, pinned_ptrs):
    n = len(pinned_ptrs)
    arr = (C.c_void_p * n)(*[_ptr(p) for p in pinned_ptrs])
    return lib().remoe_load_experts_host(h, int(layer), int(first_expert), n, arr)


def remoe_decode_step(h, hidden_in, hidden_out, selected_ids, gate_weights):
    return lib().remoe_decode_step(h, _ptr(hidden_in), _ptr(hidden_out), _ptr(selected_ids), _ptr(gate_weights))


def remoe_decode_steps(h, n_steps, hidden_in, hidden_out, selected_ids, gate_weights):
    return lib().remoe_decode_steps(h, int(n_steps), _ptr(hidden_in), _ptr(hidden_out), _ptr(selected_ids),
                                    _ptr(gate_weights))


def remoe_decode_step_chained(h, hidden_in, hidden_out, layer_inputs, selected_ids, gate_weights):
    return lib().remoe_decode_step_chained(h, _ptr(hidden_in), _ptr(hidden_out), _ptr(layer_inputs),
                                           _ptr(selected_ids), _ptr(gate_weights))


def remoe_decode_step_host(h, hidden_in, hidden_out, selected_ids, gate_weights):
    return lib().remoe_decode_step_host(h, _ptr(hidden_in), _ptr(hidden_out), _ptr(selected_ids),
                                        _ptr(gate_weights))


def remoe_last_step_trace(h, requests, hit, slot, evicted, n_unique):
    return lib().remoe_last_step_trace(h, _ptr(requests), _ptr(hit), _ptr(slot), _ptr(evicted), _ptr(n_unique))


def remoe_cache_stats(h, layer=-1):
    out = remoe_cache_counters()
    rc = lib().remoe_cache_stats(h, int(layer), C.byref(out))
    return rc, {n: int(getattr(out, n)) for n, _ in remoe_cache_counters._fields_}


def remoe_reuse_stats(h, layer=-1, last_ir=None):
    o, p = C.c_uint64(), C.c_uint64()
    rc = lib().remoe_reuse_stats(h, int(layer), C.byref(o), C.byref(p), _ptr(last_ir))
    return rc, int(o.value), int(p.value)


def remoe_cache_reset(h):
    return lib().remoe_cache_reset(h)


def remoe_set_policy(h, policy):
    return lib().remoe_set_policy(h, int(policy))


def remoe_set_reroute_beta(h, beta):
    return lib().remoe_set_reroute_beta(h, float(beta))


def remoe_set_profiling(h, on):
    return lib().remoe_set_profiling(h, int(bool(on)))


def remoe_kernel_time(h, phase):
    ms, n, b = C.c_double(), C.c_uint64(), C.c_uint64()
    rc = lib().remoe_kernel_time(h, int(phase), C.byref(ms), C.byref(n), C.byref(b))
    return rc, float(ms.value), int(n.value), int(b.value)


def remoe_launch_count(h):
    n = C.c_uint64()
    rc = lib().remoe_launch_count(h, C.byref(n))
    return rc, int(n.value)


def remoe_cache_snapshot(h, layer, expert_of_slot, stamp, use_count):
    return lib().remoe_cache_snapshot(h, int(layer), _ptr(expert_of_slot), _ptr(stamp), _ptr(use_count))


def remoe_order_check_counts(h):
    c, v = C.c_uint64(), C.c_uint64()
    rc = lib().remoe_order_check_counts(h, C.byref(c), C.byref(v))
    return rc, int(c.value), int(v.value)


def remoe_expert_ffn_static(hidden, weight_dtype, expert_blocks_dev, inter, scales, hidden_in, hidden_out,
                            cuda_stream=None):
    """Allocation-free expert sum of one layer; `expert_blocks_dev` are device tensors/addresses."""
    n = len(expert_blocks_dev)
    ptrs = (C.c_void_p * n)(*[_ptr(p) for p in expert_blocks_dev])
    inter_a = (C.c_int32 * n)(*[int(i) for i in inter])
    scales_a = (C.c_float * n)(*[float(x) for x in scales])
    return lib().remoe_expert_ffn_static(int(hidden), int(weight_dtype), n, ptrs, inter_a, scales_a,
                                         _ptr(hidden_in), _ptr(hidden_out), cuda_stream)


def remoe_reuse_mass(h, layer=-1, last_mass=None):
    m, p = C.c_double(), C.c_uint64()
    rc = lib().remoe_reuse_mass(h, int(layer), C.byref(m), C.byref(p), _ptr(last_mass))
    return rc, float(m.value), int(p.value)


def remoe_expert_load(h, layer=-1, counts=None):
    ent, cv, seen = C.c_double(), C.c_double(), C.c_int32()
    rc = lib().remoe_expert_load(h, int(layer), _ptr(counts), C.byref(ent), C.byref(cv), C.byref(seen))
    return rc, float(ent.value), float(cv.value), int(seen.value)


def remoe_step_history(h, first=0, count=None):
    n = C.c_int32()
    rc = lib().remoe_step_history(h, 0, 0, None, None, C.byref(n))
    if rc != REMOE_OK:
        return rc, None, None
    count = max(0, n.value - first) if count is None else count
    um, th = np.zeros(count, np.uint32), np.zeros(count, np.uint32)
    rc = lib().remoe_step_history(h, int(first), int(count), _ptr(um), _ptr(th), C.byref(n))
    return rc, um, th


def remoe_tpot_proxy(umiss, expert_bytes, bandwidth_gbps, batch=1, tpot_compute_ms=0.0):
    um = np.ascontiguousarray(umiss, dtype=np.uint32)
    io, pct = np.zeros(um.size, np.float64), np.zeros(3, np.float64)
    rc = lib().remoe_tpot_proxy(_ptr(um), um.size, int(expert_bytes), float(bandwidth_gbps), int(batch),
                                float(tpot_compute_ms), _ptr(io), _ptr(pct))
    return rc, io, pct


def remoe_last_cuda_error(h) -> str:
    return lib().remoe_last_cuda_error(h).decode()


def remoe_stack_destroy(h):
    lib().remoe_stack_destroy(h)


class Stack:
    """Owning convenience wrapper: raises RemoeError on any non-zero status."""

    def __init__(self, shape, cache_slots_per_layer, cuda_stream: int | None = None):
        self.shape = _shape_struct(shape)
        self.cache_slots = int(cache_slots_per_layer)
        rc, self.h = remoe_stack_create(self.shape, cache_slots_per_layer, cuda_stream)
        if rc != REMOE_OK:
            self.h = None
            raise RemoeError(rc, "remoe_stack_create")
        self._keep = []          # references that keep borrowed host blocks alive

    def _ck(self, rc, what):
        if rc != REMOE_OK:
            raise RemoeError(rc, what, remoe_last_cuda_error(self.h) if rc in (REMOE_E_CUDA, REMOE_E_DEVICE_FLAG, REMOE_E_ORDER) else "")

    def load_router(self, layer, w_router, w_shared_gate=None):
        self._ck(remoe_load_router(self.h, layer, w_router, w_shared_gate), "remoe_load_router")

    def load_shared(self, layer, idx, block):
        self._ck(remoe_load_shared(self.h, layer, idx, block), "remoe_load_shared")

    def load_experts_host(self, layer, first_expert, blocks, keep=None):
        self._ck(remoe_load_experts_host(self.h, layer, first_expert, blocks), "remoe_load_experts_host")
        self._keep.append(blocks if keep is None else keep)

    def decode_step(self, hidden_in, hidden_out, selected_ids, gate_weights):
        self._ck(remoe_decode_step(self.h, hidden_in, hidden_out, selected_ids, gate_weights), "remoe_decode_step")

    def decode_steps(self, n_steps, hidden_in, hidden_out, selected_ids, gate_weights):
        self._ck(remoe_decode_steps(self.h, n_steps, hidden_in, hidden_out, selected_ids, gate_weights),
                 "remoe_decode_steps")

    def decode_step_chained(self, hidden_in, hidden_out, layer_inputs, selected_ids, gate_weights):
        self._ck(remoe_decode_step_chained(self.h, hidden_in, hidden_out, layer_inputs, selected_ids, gate_weights),
                 "remoe_decode_step_chained")

    def decode_step_host(self, hidden_in, hidden_out, selected_ids, gate_weights):
        self._ck(remoe_decode_step_host(self.h, hidden_in, hidden_out, selected_ids, gate_weights),
                 "remoe_decode_step_host")

    def last_step_trace(self):
        L, BK = self.shape.n_layers, self.shape.batch * self.shape.top_k
        req, hit, slot, ev = (np.empty((L, BK), np.int32) for _ in range(4))
        nu = np.empty(L, np.int32)
        self._ck(remoe_last_step_trace(self.h, req, hit, slot, ev, nu), "remoe_last_step_trace")
        return dict(requests=req, hit=hit, slot=slot, evicted=ev, n_unique=nu)

    def cache_stats(self, layer=-1):
        rc, out = remoe_cache_stats(self.h, layer)
        self._ck(rc, "remoe_cache_stats")
        return out

    def reuse_stats(self, layer=-1, want_last_ir=False):
        n = self.shape.batch * (self.shape.n_layers if layer < 0 else 1)
        ir = np.empty(n, np.float32) if want_last_ir else None
        rc, o, p = remoe_reuse_stats(self.h, layer, ir)
        self._ck(rc, "remoe_reuse_stats")
        return (o, p, ir) if want_last_ir else (o, p)

    def reuse_mass(self, layer=-1, want_last=False):
        n = self.shape.batch * (self.shape.n_layers if layer < 0 else 1)
        last = np.empty(n, np.float32) if want_last else None
        rc, m, p = remoe_reuse_mass(self.h, layer, last)
        self._ck(rc, "remoe_reuse_mass")
        return (m, p, last) if want_last else (m, p)

    def expert_load(self, layer=-1):
        """(counts [L, N] or [N] uint64, normalised entropy, CV, experts visited)."""
        n = self.shape.n_routed * (self.shape.n_layers if layer < 0 else 1)
        counts = np.zeros(n, np.uint64)
        rc, ent, cv, seen = remoe_expert_load(self.h, layer, counts)
        self._ck(rc, "remoe_expert_load")
        return (counts.reshape(-1, self.shape.n_routed) if layer < 0 else counts), ent, cv, seen

    def step_history(self, first=0, count=None):
        rc, um, th = remoe_step_history(self.h, first, count)
        self._ck(rc, "remoe_step_history")
        return um, th

    def cache_reset(self):
        self._ck(remoe_cache_reset(self.h), "remoe_cache_reset")

    def set_policy(self, policy):
        self._ck(remoe_set_policy(self.h, policy), "remoe_set_policy")

    def set_reroute_beta(self, beta):
        self._ck(remoe_set_reroute_beta(self.h, beta), "remoe_set_reroute_beta")

    def set_profiling(self, on):
        self._ck(remoe_set_profiling(self.h, on), "remoe_set_profiling")

    def kernel_time(self, phase):
        rc, ms, n, b = remoe_kernel_time(self.h, phase)
        self._ck(rc, "remoe_kernel_time")
        return ms, n, b

    def launch_count(self):
        rc, n = remoe_launch_count(self.h)
        self._ck(rc, "remoe_launch_count")
        return n

    def cache_snapshot(self, layer):
        """(expert_of_slot [C] int32, stamp [C] uint64, use_count [C] uint32) of one layer."""
        eos = np.empty(self.cache_slots, np.int32)
        stamp = np.empty(self.cache_slots, np.uint64)
        freq = np.empty(self.cache_slots, np.uint32)
        self._ck(remoe_cache_snapshot(self.h, layer, eos, stamp, freq), "remoe_cache_snapshot")
        return eos, stamp, freq

    def order_check_counts(self):
        rc, c, v = remoe_order_check_counts(self.h)
        self._ck(rc, "remoe_order_check_counts")
        return c, v

    def close(self):
        if self.h is not None:
            remoe_stack_destroy(self.h)
            self.h = None
            self._keep = []

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
