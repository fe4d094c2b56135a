"""Seeded synthetic workloads: shapes, weight tensors and hidden-state streams.

Every tensor is a pure function of (seed, tensor kind, layer, index) through numpy's
counter-based Philox generator, so a single expert or a single decode step can be
regenerated in isolation and two consumers always see identical bytes.

Storage conventions produced here (they are data layouts, not arithmetic):

* router weights      ``[N, H]`` row-major, one row per routed expert;
* shared-gate vector  ``[H]``;
* expert block        ``[I, 3, H]`` row-major: for intermediate index ``i`` the three
  consecutive rows are ``W_gate[i, :]``, ``W_up[i, :]`` and ``W_down[:, i]`` (column ``i``
  of the down projection), so that everything needed for one intermediate channel is one
  contiguous run of ``3*H`` elements;
* hidden states       ``[L, B, H]`` float32 per decode step.

Element type is float32 (``weight_dtype == 0``) or bfloat16 stored as ``uint16`` bit
patterns (``weight_dtype == 1``), rounded to nearest-even once, at generation.  With
``weight_dtype == 2`` the expert blocks are OCP FP8 E4M3 bytes whose value is
``decode(byte) * 2**-FP8_SHIFT`` (a fixed power-of-two scale that puts N(0, 0.02^2) weights in
the format's normal range) while the router and shared-gate weights stay bfloat16.  With
``weight_dtype == 3`` the expert blocks are 4-bit integers in groups of 32 consecutive elements of a
row with one bfloat16 scale per group (see ``int4_g32_encode``); router and shared gate again bfloat16.
"""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, asdict
import os

import numpy as np

KIND_ROUTER = 1
KIND_SHARED_GATE = 2
KIND_EXPERT = 3
KIND_SHARED = 4
KIND_HIDDEN = 5
KIND_RHO = 6

EXPERT_STD = 0.02
FP8_SHIFT = 8
INT4_GROUP = 32


@dataclass(frozen=True)
class Shape:
    n_layers: int
    hidden: int
    n_routed: int
    top_k: int
    inter_routed: int
    n_shared: int = 0
    inter_shared: int = 0
    shared_gate: int = 0      # 1: shared output scaled by sigmoid(w_sg . h)
    renorm_topk: int = 0      # 1: top-k gate weights renormalised to sum to 1
    weight_dtype: int = 0     # 0 float32, 1 bfloat16, 2 fp8 e4m3, 3 int4 in groups of 32
    batch: int = 1

    def asdict(self):
        return asdict(self)

    @property
    def elem_bytes(self) -> int:
        """Bytes per element of an expert block (whole-byte formats only)."""
        return {0: 4, 1: 2, 2: 1}[self.weight_dtype]

    @property
    def row_bytes(self) -> int:
        """Bytes of one stored row of `hidden` expert-block elements."""
        if self.weight_dtype == 3:
            return self.hidden // 2 + 2 * (self.hidden // INT4_GROUP)
        return self.hidden * self.elem_bytes

    @property
    def router_dtype(self) -> int:
        """Element type of router and shared-gate weights (fp8 stacks keep them in bf16)."""
        return 0 if self.weight_dtype == 0 else 1


# The five workloads; `rhos` lists the AR(1) coefficients swept for that workload
# (None = one coefficient per sequence drawn U(0.3, 0.95) from the seed).
CONFIGS = {
    "tiny_fp32": dict(
        shape=Shape(1, 256, 16, 2, 128, 0, 0, 0, 0, 0, 1),
        cache_slots=4, steps=64, rhos=(0.9,), seed=0),
    "dsv2lite": dict(
        shape=Shape(26, 2048, 64, 6, 1408, 2, 1408, 0, 0, 1, 1),
        cache_slots=16, steps=512, rhos=(0.0, 0.5, 0.9), seed=0),
    "qwen15moe": dict(
        shape=Shape(24, 2048, 60, 4, 1408, 1, 5632, 1, 0, 1, 1),
        cache_slots=12, steps=512, rhos=(0.8,), seed=0),
    "qwen3_30b": dict(
        shape=Shape(48, 2048, 128, 8, 768, 0, 0, 0, 1, 1, 1),
        cache_slots=32, steps=1024, rhos=(0.5, 0.9), seed=0),
    "dsv2lite_fp8": dict(
        shape=Shape(26, 2048, 64, 6, 1408, 2, 1408, 0, 0, 2, 1),
        cache_slots=16, steps=512, rhos=(0.9, 0.5, 0.0), seed=0),
    "dsv2lite_int4": dict(
        shape=Shape(26, 2048, 64, 6, 1408, 2, 1408, 0, 0, 3, 1),
        cache_slots=16, steps=512, rhos=(0.9, 0.5, 0.0), seed=0),
    "dsv2lite_b32": dict(
        shape=Shape(26, 2048, 64, 6, 1408, 2, 1408, 0, 0, 1, 32),
        cache_slots=32, steps=1024, rhos=(None,), seed=0),
    "dsv2lite_b32_int4": dict(
        shape=Shape(26, 2048, 64, 6, 1408, 2, 1408, 0, 0, 3, 32),
        cache_slots=32, steps=1024, rhos=(None,), seed=0),
    "dsv2lite_b32_fp8": dict(
        shape=Shape(26, 2048, 64, 6, 1408, 2, 1408, 0, 0, 2, 32),
        cache_slots=32, steps=1024, rhos=(None,), seed=0),
}


def config(name: str) -> dict:
    return dict(CONFIGS[name])


def expert_block_elems(hidden: int, inter: int) -> int:
    return 3 * hidden * inter


def expert_block_bytes(shape: Shape, shared: bool = False) -> int:
    inter = shape.inter_shared if shared else shape.inter_routed
    return 3 * inter * shape.row_bytes


def bf16_round_to_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 bit patterns (uint16), round to nearest, ties to even."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    return ((u + np.uint32(0x7FFF) + lsb) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """bfloat16 bit patterns (uint16) -> the float32 values they denote (exact)."""
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def _fp8_table() -> np.ndarray:
    """The 256 values of OCP FP8 E4M3: 1 sign, 4 exponent (bias 7), 3 mantissa bits; exponent 0 is
    subnormal (m/8 * 2^-6); there are no infinities and S.1111.111 is NaN; largest finite 448."""
    t = np.zeros(256, dtype=np.float32)
    for b in range(256):
        sgn = -1.0 if b & 0x80 else 1.0
        e, m = (b >> 3) & 0xF, b & 7
        if e == 0xF and m == 7:
            t[b] = np.nan
        elif e == 0:
            t[b] = sgn * (m / 8.0) * 2.0 ** -6
        else:
            t[b] = sgn * (1.0 + m / 8.0) * 2.0 ** (e - 7)
    return t


_FP8 = _fp8_table()


def fp8_e4m3_round_to_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> FP8 E4M3 bytes: nearest value, ties to the even code, magnitudes above 448 saturate.

    Done on the bit patterns: in the normal range (|x| >= 2^-6) the 23-bit mantissa is rounded to 3 bits,
    nearest even, with the carry running into the exponent, and the exponent is re-biased from 127 to 7;
    below that the format is subnormal, multiples of 2^-9, and |x| * 2^9 is rounded to an integer."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    a = u & np.uint32(0x7FFFFFFF)
    r = (a + np.uint32(0x7FFFF) + ((a >> np.uint32(20)) & np.uint32(1))) >> np.uint32(20)
    code = r.astype(np.int32) - ((127 - 7) << 3)
    small = a < np.uint32(0x3C800000)                                   # |x| < 2^-6
    sub = np.rint(np.minimum(a.view(np.float32), np.float32(1.0)) * np.float32(512.0)).astype(np.int32)
    code = np.clip(np.where(small, sub, code), 0, 126).astype(np.uint8)
    return code | ((u >> np.uint32(24)) & np.uint32(0x80)).astype(np.uint8)


def fp8_e4m3_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """FP8 E4M3 bytes -> the float32 values they denote (exact), without the stack-wide scale."""
    return _FP8[np.asarray(bits, dtype=np.uint8)]


def int4_g32_encode(x: np.ndarray, hidden: int) -> np.ndarray:
    """float32 rows of `hidden` elements -> the 4-bit grouped storage format, as bytes.

    Each row is cut into groups of 32 consecutive elements.  A group's scale is max|x| / 7 rounded to
    bfloat16 (nearest, ties to even); its codes are q = round-half-even(x / scale) clipped to [-7, 7]
    (all zero when the scale is zero), stored offset by 8 as unsigned nibbles, element 2i in the low and
    element 2i+1 in the high half of byte i.  A stored row is `hidden/2` bytes of codes followed by
    `hidden/32` bfloat16 scales (little endian); rows follow each other without padding.  The value a
    stored element denotes is (nibble - 8) * scale."""
    x = np.ascontiguousarray(x, dtype=np.float32).reshape(-1, hidden // INT4_GROUP, INT4_GROUP)
    rows = x.shape[0]
    amax = np.max(np.abs(x), axis=2)
    s_bits = bf16_round_to_bits((amax / np.float32(7.0)).astype(np.float32))
    s = bf16_bits_to_f32(s_bits)
    safe = np.where(s > 0, s, np.float32(1.0))
    q = np.clip(np.rint(x / safe[:, :, None]), -7, 7).astype(np.int16)
    q = np.where(s[:, :, None] > 0, q, 0)
    u = (q + 8).astype(np.uint8).reshape(rows, hidden)
    packed = (u[:, 0::2] | (u[:, 1::2] << 4)).astype(np.uint8)
    out = np.empty((rows, hidden // 2 + 2 * (hidden // INT4_GROUP)), dtype=np.uint8)
    out[:, :hidden // 2] = packed
    out[:, hidden // 2:] = s_bits.astype("<u2").view(np.uint8).reshape(rows, -1)
    return out.reshape(-1)


def int4_g32_decode(b: np.ndarray, hidden: int) -> np.ndarray:
    """Bytes in the 4-bit grouped format -> the float32 values they denote (exact), flattened row by row."""
    row = hidden // 2 + 2 * (hidden // INT4_GROUP)
    b = np.asarray(b, dtype=np.uint8).reshape(-1, row)
    codes = b[:, :hidden // 2]
    u = np.empty((b.shape[0], hidden), dtype=np.int16)
    u[:, 0::2] = codes & 0xF
    u[:, 1::2] = codes >> 4
    s = bf16_bits_to_f32(np.ascontiguousarray(b[:, hidden // 2:]).view("<u2").astype(np.uint16))
    v = (u - 8).astype(np.float32).reshape(b.shape[0], -1, INT4_GROUP) * s[:, :, None]
    return v.reshape(-1)


def widen(shape: "Shape", a: np.ndarray, router: bool = False) -> np.ndarray:
    """Stored weights -> the float32 values they denote (router=True for router / gate tensors)."""
    dt = shape.router_dtype if router else shape.weight_dtype
    if dt == 1:
        return bf16_bits_to_f32(a)
    if dt == 2:
        return fp8_e4m3_bits_to_f32(a) * np.float32(2.0 ** -FP8_SHIFT)
    if dt == 3:
        return int4_g32_decode(a, shape.hidden)
    return a


def _rng(seed: int, kind: int, a: int = 0, b: int = 0) -> np.random.Generator:
    key = np.array([(int(seed) << 32) | int(kind), (int(a) << 32) | int(b)], dtype=np.uint64)
    return np.random.Generator(np.random.Philox(key=key))


def _store(x32: np.ndarray, weight_dtype: int, out: np.ndarray | None, hidden: int = 0) -> np.ndarray:
    if weight_dtype == 3:
        bits = int4_g32_encode(x32, hidden)
        if out is None:
            return bits
        out[...] = bits.reshape(out.shape)
        return out
    if weight_dtype == 2:
        bits = fp8_e4m3_round_to_bits(x32 * np.float32(2.0 ** FP8_SHIFT))
        if out is None:
            return bits
        out[...] = bits.reshape(out.shape)
        return out
    if weight_dtype == 1:
        bits = bf16_round_to_bits(x32)
        if out is None:
            return bits
        out[...] = bits.reshape(out.shape)
        return out
    if out is None:
        return x32
    out[...] = x32.reshape(out.shape)
    return out


def gen_router(seed: int, shape: Shape, layer: int) -> np.ndarray:
    """Router weights [N, H], entries N(0, 1/H)."""
    g = _rng(seed, KIND_ROUTER, layer)
    x = g.standard_normal((shape.n_routed, shape.hidden), dtype=np.float32)
    x *= np.float32(1.0 / np.sqrt(shape.hidden))
    return _store(x, shape.router_dtype, None)


def gen_shared_gate(seed: int, shape: Shape, layer: int) -> np.ndarray:
    """Shared-expert gate vector [H], entries N(0, 1/H)."""
    g = _rng(seed, KIND_SHARED_GATE, layer)
    x = g.standard_normal((shape.hidden,), dtype=np.float32)
    x *= np.float32(1.0 / np.sqrt(shape.hidden))
    return _store(x, shape.router_dtype, None)


def gen_expert_block(seed: int, shape: Shape, layer: int, expert: int,
                     out: np.ndarray | None = None) -> np.ndarray:
    """Routed expert block [I, 3, H] (flattened), entries N(0, 0.02^2)."""
    n = expert_block_elems(shape.hidden, shape.inter_routed)
    g = _rng(seed, KIND_EXPERT, layer, expert)
    x = g.standard_normal((n,), dtype=np.float32)
    x *= np.float32(EXPERT_STD)
    return _store(x, shape.weight_dtype, out, shape.hidden)


def gen_shared_block(seed: int, shape: Shape, layer: int, idx: int,
                     out: np.ndarray | None = None) -> np.ndarray:
    """Shared expert block [I_s, 3, H] (flattened), entries N(0, 0.02^2)."""
    n = expert_block_elems(shape.hidden, shape.inter_shared)
    g = _rng(seed, KIND_SHARED, layer, idx)
    x = g.standard_normal((n,), dtype=np.float32)
    x *= np.float32(EXPERT_STD)
    return _store(x, shape.weight_dtype, out, shape.hidden)


def fill_expert_store(seed: int, shape: Shape, store: np.ndarray, layers=None,
                      threads: int | None = None) -> None:
    """Fill ``store[L, N, 3*I*H]`` (a view over caller-owned, e.g. pinned, memory)."""
    layers = range(shape.n_layers) if layers is None else layers
    jobs = [(l, e) for l in layers for e in range(shape.n_routed)]
    threads = threads or len(os.sched_getaffinity(0))

    def one(le):
        l, e = le
        gen_expert_block(seed, shape, l, e, out=store[l, e])

    if threads <= 1 or len(jobs) < 4:
        for j in jobs:
            one(j)
    else:
        with ThreadPoolExecutor(threads) as ex:
            list(ex.map(one, jobs))


def expert_matrices(block: np.ndarray, hidden: int, inter: int):
    """Views (W_gate [I,H], W_up [I,H], W_down [H,I]) into a packed expert block."""
    b = block.reshape(inter, 3, hidden)
    return b[:, 0, :], b[:, 1, :], b[:, 2, :].T


class HiddenStream:
    """Per-layer, per-sequence AR(1) hidden states, one ``[L, B, H]`` array per step.

    ``h_1 = eps_1`` and ``h_t = rho * h_{t-1} + sqrt(1 - rho^2) * eps_t`` with
    ``eps ~ N(0, I)`` independent per (step, layer, sequence); everything in float32.
    ``rho`` is a scalar, or ``None`` for one coefficient per sequence drawn U(0.3, 0.95).
    """

    def __init__(self, seed: int, shape: Shape, rho):
        self.seed, self.shape = seed, shape
        B = shape.batch
        if rho is None:
            r = _rng(seed, KIND_RHO).uniform(0.3, 0.95, size=B)
        else:
            r = np.full(B, float(rho))
        self.rho = r.astype(np.float32)
        self._a = self.rho.reshape(1, B, 1)
        self._c = np.sqrt(np.float32(1.0) - self.rho * self.rho).astype(np.float32).reshape(1, B, 1)
        self.t = 0
        self._h = None

    def step(self) -> np.ndarray:
        s = self.shape
        eps = _rng(self.seed, KIND_HIDDEN, self.t).standard_normal(
            (s.n_layers, s.batch, s.hidden), dtype=np.float32)
        if self._h is None:
            self._h = eps
        else:
            self._h = (self._a * self._h + self._c * eps).astype(np.float32)
        self.t += 1
        return self._h

    def take(self, n_steps: int) -> np.ndarray:
        """Next ``n_steps`` states as ``[n_steps, L, B, H]`` float32."""
        s = self.shape
        out = np.empty((n_steps, s.n_layers, s.batch, s.hidden), dtype=np.float32)
        for i in range(n_steps):
            out[i] = self.step()
        return out
