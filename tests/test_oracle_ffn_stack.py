"""Pins for the oracle's expert arithmetic and for the stepped stack (counters, reuse)."""
import math

import numpy as np
import pytest
import torch

from oracle import remoe_oracle as orc
import synth


def test_silu_values():
    assert orc.silu(0.0) == 0.0
    assert abs(float(orc.silu(1.0)) - 0.7310585786300049) < 1e-15      # 1 / (1 + e^-1)
    assert abs(float(orc.silu(-1.0)) + 0.2689414213699951) < 1e-15     # -1 / (1 + e)
    assert abs(float(orc.silu(40.0)) - 40.0) < 1e-12
    x = np.linspace(-6, 6, 25)
    assert np.allclose(orc.silu(x) - orc.silu(-x), x, atol=1e-14)       # silu(x) - silu(-x) = x


def test_expert_hand_example():
    # H = 2, I = 1: y = W_down[:, 0] * silu(x_0) * x_1
    wg = np.array([[1.0, 0.0]]); wu = np.array([[0.0, 1.0]]); wd = np.array([[2.0], [3.0]])
    x = np.array([0.7, -1.5])
    a = (0.7 / (1 + math.exp(-0.7))) * -1.5
    assert np.allclose(orc.swiglu_expert(wg, wu, wd, x), [2 * a, 3 * a], rtol=1e-15)


def test_single_expert_matches_library_ops():
    """N = K = 1: the gate weight is exactly 1 and the layer is one SwiGLU expert, which
    torch evaluates with its own silu and matmul."""
    rng = np.random.default_rng(0)
    H, I = 48, 20
    wg, wu, wd = rng.standard_normal((I, H)), rng.standard_normal((I, H)), rng.standard_normal((H, I))
    wr = rng.standard_normal((1, H))
    x = rng.standard_normal(H)
    z = orc.router_logits(wr, x)
    ids, _ = orc.topk_select(z, 1)
    g = orc.gate_weights(orc.softmax(z), ids, False)
    assert g[0] == 1.0
    out = orc.moe_output(x, ids, g, 1, lambda e: (wg, wu, wd))
    tx = torch.from_numpy(x)
    ref = torch.from_numpy(wd) @ (torch.nn.functional.silu(torch.from_numpy(wg) @ tx) * (torch.from_numpy(wu) @ tx))
    assert np.allclose(out, ref.numpy(), rtol=1e-12, atol=1e-12)


def _toy(seed, n=6, H=16, I=8):
    rng = np.random.default_rng(seed)
    ws = [(rng.standard_normal((I, H)), rng.standard_normal((I, H)), rng.standard_normal((H, I)))
          for _ in range(n)]
    return ws, rng.standard_normal(H)


def test_dense_equals_selected_and_masking():
    ws, x = _toy(1)
    ids, g = [4, 1, 3], [0.5, 0.25, 0.125]
    d = orc.moe_output(x, ids, g, 6, lambda e: ws[e], mode="dense")
    s = orc.moe_output(x, ids, g, 6, lambda e: ws[e], mode="selected")
    assert np.array_equal(d, s)
    by_hand = 0.25 * orc.swiglu_expert(*ws[1], x) + 0.125 * orc.swiglu_expert(*ws[3], x) \
        + 0.5 * orc.swiglu_expert(*ws[4], x)
    assert np.allclose(d, by_hand, rtol=1e-13, atol=1e-13)


def test_linearity_zero_and_shared():
    ws, x = _toy(2)
    ids = [0, 5]
    y0, y5 = orc.swiglu_expert(*ws[0], x), orc.swiglu_expert(*ws[5], x)
    a = orc.moe_output(x, ids, [0.3, 0.6], 6, lambda e: ws[e])
    b = orc.moe_output(x, ids, [0.6, 1.2], 6, lambda e: ws[e])
    assert np.allclose(2 * a, b, rtol=1e-13)
    assert np.allclose(a, 0.3 * y0 + 0.6 * y5, rtol=1e-13)
    zero = (np.zeros((8, 16)), np.zeros((8, 16)), np.zeros((16, 8)))
    assert np.array_equal(orc.moe_output(x, [0], [1.0], 1, lambda e: zero), np.zeros(16))
    sh = orc.moe_output(x, ids, [0.3, 0.6], 6, lambda e: ws[e], shared_weights=[ws[2], ws[3]])
    assert np.allclose(sh - a, orc.swiglu_expert(*ws[2], x) + orc.swiglu_expert(*ws[3], x), rtol=1e-12, atol=1e-12)
    sh2 = orc.moe_output(x, ids, [0.3, 0.6], 6, lambda e: ws[e], shared_weights=[ws[2]], shared_scale=0.25)
    assert np.allclose(sh2 - a, 0.25 * orc.swiglu_expert(*ws[2], x), rtol=1e-12, atol=1e-12)
    assert orc.sigmoid(0.0) == 0.5 and abs(orc.sigmoid(2.0) + orc.sigmoid(-2.0) - 1.0) < 1e-15


# ------------------------------------------------------------------------------- stack

def _stack(shape, cache_slots, seed=0, with_ffn=False, policy="lru"):
    routers = [synth.gen_router(seed, shape, l) for l in range(shape.n_layers)]
    sg = [synth.gen_shared_gate(seed, shape, l) for l in range(shape.n_layers)] if shape.shared_gate else None
    if shape.weight_dtype == 1:
        routers = [synth.bf16_bits_to_f32(r) for r in routers]
        sg = None if sg is None else [synth.bf16_bits_to_f32(v) for v in sg]

    def widen(b):
        return synth.bf16_bits_to_f32(b) if shape.weight_dtype == 1 else b

    def ew(l, e):
        return synth.expert_matrices(widen(synth.gen_expert_block(seed, shape, l, e)), shape.hidden, shape.inter_routed)

    def sw(l, i):
        return synth.expert_matrices(widen(synth.gen_shared_block(seed, shape, l, i)), shape.hidden, shape.inter_shared)

    return orc.OracleStack(shape, cache_slots, routers, ew if with_ffn else None, sw if with_ffn else None,
                           shared_gates=sg, policy=policy)


def test_tiny_config_invariants():
    cfg = synth.config("tiny_fp32")
    shape = cfg["shape"]
    st = _stack(shape, cfg["cache_slots"], with_ffn=True)
    hs = synth.HiddenStream(0, shape, 0.9)
    T = cfg["steps"]
    prev_ids = None
    for t in range(T):
        h = hs.step()
        r = st.step(h, ffn="dense" if t < 4 else "selected")
        if t < 4:
            st2 = orc.moe_output(h[0, 0], r["ids"][0, 0], r["gates"][0, 0], shape.n_routed,
                                 lambda e: st.expert_weights(0, e), mode="selected")
            assert np.array_equal(st2, r["out"][0, 0])
        assert r["gates"][0, 0].sum() <= 1.0 + 1e-12
        ov = r["overlap"][0, 0]
        if t == 0:
            assert ov == -1 and sum(r["hit"][0]) == 0
        else:
            assert 0 <= ov <= shape.top_k
            assert ov == len(set(r["ids"][0, 0]) & set(prev_ids))
            assert len(r["hit"][0]) - sum(r["hit"][0]) <= shape.top_k - ov       # Prop. 3.1
        prev_ids = r["ids"][0, 0]
    assert st.tok_hits[0] + st.tok_misses[0] == shape.n_layers * shape.top_k * T
    assert st.uniq_hits == st.tok_hits and st.uniq_misses == st.tok_misses       # B = 1: dedup is a no-op
    assert st.pairs_counted[0] == T - 1
    assert 0.0 <= st.eor() <= 1.0 and 0.0 <= st.uhr() <= 1.0


def test_constant_stream_reuses_everything():
    shape = synth.Shape(2, 64, 12, 3, 8)
    st = _stack(shape, 3)
    h = np.random.default_rng(0).standard_normal((2, 1, 64)).astype(np.float32)
    for t in range(10):
        r = st.step(h, ffn=None)
        if t:
            assert (r["overlap"] == 3).all() and all(all(x) for x in r["hit"])
    assert st.eor() == 1.0 and sum(st.uniq_misses) == 2 * 3


def test_layers_are_independent():
    shape = synth.Shape(3, 64, 16, 2, 8)
    full = _stack(shape, 4)
    hs = synth.HiddenStream(1, shape, 0.7).take(40)
    traces = [full.step(hs[t], ffn=None) for t in range(40)]
    for l in range(3):
        one = orc.OracleStack(synth.Shape(1, 64, 16, 2, 8), 4, [full.routers[l]])
        for t in range(40):
            r = one.step(hs[t, l:l + 1], ffn=None)
            assert np.array_equal(r["ids"][0], traces[t]["ids"][l])
            assert r["hit"][0] == traces[t]["hit"][l] and r["slot"][0] == traces[t]["slot"][l]
        assert one.uniq_misses[0] == full.uniq_misses[l]
    assert sum(full.uniq_misses) == sum(len(tr["hit"][l]) - sum(tr["hit"][l]) for tr in traces for l in range(3))


def test_batched_counters():
    shape = synth.Shape(2, 64, 16, 3, 8, batch=5)
    st = _stack(shape, 8)
    hs = synth.HiddenStream(2, shape, None)
    T, sum_u = 30, 0
    for t in range(T):
        before = [c.resident() for c in st.caches]
        th0 = list(st.tok_hits)
        r = st.step(hs.step(), ffn=None)
        for l in range(2):
            flat = [int(e) for e in r["ids"][l].reshape(-1)]
            assert r["requests"][l] == orc.unique_in_order(flat)
            assert st.tok_hits[l] - th0[l] == sum(1 for e in flat if e in before[l])
            assert r["hit"][l] == [e in before[l] for e in r["requests"][l]]
            sum_u += len(r["requests"][l])
    assert sum(st.tok_hits) + sum(st.tok_misses) == 2 * 5 * 3 * T
    assert sum(st.uniq_hits) + sum(st.uniq_misses) == sum_u
    assert st.pairs_counted == [(T - 1) * 5] * 2


def test_iid_stream_statistics():
    """rho = 0: consecutive selections are independent, so EOR is near K/N and, for
    exchangeable experts, the LRU hit rate is near C/N (loose statistical check)."""
    shape = synth.Shape(4, 64, 32, 4, 8)
    st = _stack(shape, 8)
    hs = synth.HiddenStream(3, shape, 0.0)
    for _ in range(400):
        st.step(hs.step(), ffn=None)
    assert abs(st.eor() - 4 / 32) < 0.03
    assert abs(st.uhr() - 8 / 32) < 0.06


def test_id_override_and_reset():
    shape = synth.Shape(1, 64, 16, 2, 8)
    st = _stack(shape, 4)
    h = synth.HiddenStream(4, shape, 0.5).take(3)
    r0 = st.step(h[0], ffn=None)
    forced = [int(r0["ids"][0, 0][0]), 15 if 15 not in r0["ids"][0, 0] else 14]
    r1 = st.step(h[1], ffn=None, id_override={(0, 0): forced})
    assert list(r1["ids"][0, 0]) == forced and r1["requests"][0] == forced
    assert r1["hit"][0][0] is True
    st.reset()
    assert st.caches[0].resident() == set() and st.pairs_counted == [0]
    r2 = st.step(h[0], ffn=None)
    assert np.array_equal(r2["ids"], r0["ids"]) and sum(r2["hit"][0]) == 0 and r2["overlap"][0, 0] == -1


def test_synth_is_reproducible_and_layout():
    shape = synth.Shape(2, 32, 4, 2, 6, weight_dtype=1)
    a = synth.gen_expert_block(0, shape, 1, 3)
    b = synth.gen_expert_block(0, shape, 1, 3)
    assert a.dtype == np.uint16 and np.array_equal(a, b) and a.size == 3 * 32 * 6
    assert not np.array_equal(a, synth.gen_expert_block(0, shape, 1, 2))
    wg, wu, wd = synth.expert_matrices(a, 32, 6)
    assert wg.shape == (6, 32) and wd.shape == (32, 6)
    blk = a.reshape(6, 3, 32)
    assert np.array_equal(wg[2], blk[2, 0]) and np.array_equal(wu[2], blk[2, 1]) and np.array_equal(wd[:, 2], blk[2, 2])
    x = np.array([1.0, 1.00390625, -2.5, 3.0e-3], dtype=np.float32)       # 1.00390625 = 1 + 2^-8: tie -> even
    bits = synth.bf16_round_to_bits(x)
    assert bits[0] == 0x3F80 and bits[1] == 0x3F80
    back = synth.bf16_bits_to_f32(bits)
    assert np.all(np.abs(back - x) <= np.abs(x) * 2.0 ** -8)
    hs1 = synth.HiddenStream(5, shape, 0.9).take(5)
    hs2 = synth.HiddenStream(5, shape, 0.9).take(5)
    assert np.array_equal(hs1, hs2) and hs1.shape == (5, 2, 1, 32)
    long = synth.HiddenStream(6, synth.Shape(1, 4096, 4, 2, 6), 0.9).take(200)[:, 0, 0]
    c = np.mean(long[1:] * long[:-1]) / np.mean(long * long)
    assert abs(c - 0.9) < 0.02 and abs(long.std() - 1.0) < 0.05


def test_chained_mode_identities():
    """x_l = rmsnorm(h_l), h_{l+1} = h_l + MoE_l(x_l): telescoping sum, agreement with one-layer stacks run by hand, and
    the zero-weight case where every layer sees h_0."""
    shape = synth.Shape(3, 64, 8, 2, 8, 1, 8)
    st = _stack(shape, 3, seed=9, with_ffn=True)
    h0 = np.random.default_rng(9).standard_normal((1, 64))
    r = st.step(h0, ffn="dense", chained=True)
    assert np.allclose(r["final"] - h0, r["out"].sum(axis=0), rtol=1e-13, atol=1e-13)
    for l in range(2):
        assert np.allclose(r["layer_inputs"][l + 1] - r["layer_inputs"][l], r["out"][l], rtol=1e-13, atol=1e-13)
    assert np.array_equal(r["layer_inputs"][0], h0)
    cur = h0.copy()
    for l in range(3):
        one = orc.OracleStack(synth.Shape(1, 64, 8, 2, 8, 1, 8), 3, [st.routers[l]],
                              lambda _l, e, l=l: st.expert_weights(l, e), lambda _l, i, l=l: st.shared_weights(l, i))
        x = cur / np.sqrt((cur ** 2).sum() / 64 + 1e-6)                # pre-norm, unit RMS
        assert abs(np.sqrt((x ** 2).mean()) - 1.0) < 1e-5
        r1 = one.step(x[None], ffn="selected")
        assert np.array_equal(r1["ids"][0], r["ids"][l])
        assert np.allclose(r1["out"][0], r["out"][l], rtol=1e-13, atol=1e-13)
        cur = cur + r1["out"][0]
    assert np.allclose(cur, r["final"], rtol=1e-13, atol=1e-13)

    zero = (np.zeros((8, 64)), np.zeros((8, 64)), np.zeros((64, 8)))
    stz = orc.OracleStack(shape, 3, st.routers, lambda l, e: zero, lambda l, i: zero)
    rz = stz.step(h0, ffn="selected", chained=True)
    assert np.array_equal(rz["final"], h0) and all(np.array_equal(x, h0) for x in rz["layer_inputs"])
    x0 = h0 / np.sqrt((h0 ** 2).mean() + 1e-6)
    plain = orc.OracleStack(shape, 3, st.routers).step(np.repeat(x0[None], 3, axis=0), ffn=None)
    assert np.array_equal(plain["ids"], rz["ids"])


def test_fp8_storage_matches_library_cast():
    """FP8 E4M3 bytes of the generator against torch's float8_e4m3fn: decode of all 256 codes and
    round-to-nearest-even encode of in-range values; larger magnitudes saturate at 448."""
    codes = np.arange(256, dtype=np.uint8)
    ours = synth.fp8_e4m3_bits_to_f32(codes)
    ref = torch.from_numpy(codes).view(torch.float8_e4m3fn).to(torch.float32).numpy()
    assert np.array_equal(np.isnan(ours), np.isnan(ref)) and np.array_equal(ours[~np.isnan(ours)], ref[~np.isnan(ref)])
    x = np.random.default_rng(0).standard_normal(100000).astype(np.float32) * 5.12
    x = np.concatenate([x, np.array([0.0, 448.0, 17.0, 18.0, 19.0, 2.0 ** -10, -2.0 ** -10, 0.0009], np.float32)])
    ref_bits = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(synth.fp8_e4m3_round_to_bits(x), ref_bits)
    assert list(synth.fp8_e4m3_round_to_bits(np.array([1000.0, -1000.0], np.float32))) == [126, 254]
    # every midpoint between neighbouring codes goes to the even code, its float32 neighbours to either side
    vals = synth.fp8_e4m3_bits_to_f32(np.arange(127, dtype=np.uint8)).astype(np.float64)
    mids = ((vals[1:] + vals[:-1]) / 2).astype(np.float32)
    lo = np.arange(126)
    assert np.array_equal(synth.fp8_e4m3_round_to_bits(mids), np.where(lo % 2 == 0, lo, lo + 1).astype(np.uint8))
    assert np.array_equal(synth.fp8_e4m3_round_to_bits(np.nextafter(mids, np.float32(0))), lo.astype(np.uint8))
    assert np.array_equal(synth.fp8_e4m3_round_to_bits(np.nextafter(mids, np.float32(1e9))), (lo + 1).astype(np.uint8))
    assert np.array_equal(synth.fp8_e4m3_round_to_bits(-mids), (np.where(lo % 2 == 0, lo, lo + 1) | 0x80).astype(np.uint8))
    shape = synth.Shape(1, 512, 4, 2, 8, 0, 0, 0, 0, 2, 1)
    blk = synth.gen_expert_block(0, shape, 0, 1)
    assert blk.dtype == np.uint8 and synth.gen_router(0, shape, 0).dtype == np.uint16
    w = synth.widen(shape, blk)
    assert 0.015 < w.std() < 0.025 and np.abs(w).max() < 448 / 256


def test_int4_grouped_storage_hand_example_and_error_bound():
    """The 4-bit grouped format against a group worked by hand and against its definition: value =
    (code - 8) * bf16 scale, scale = bf16(max|x| / 7), codes = round-half-even(x / scale) in [-7, 7];
    a row is H/2 code bytes (element 2i in the low half of byte i) followed by H/32 little-endian bf16
    scales."""
    H = 64
    x = np.zeros((2, H), np.float32)
    # row 0, group 0: max 3.5 -> scale 0.5 exactly; codes = x / 0.5
    x[0, :8] = [3.5, -3.5, 0.5, -0.5, 0.25, 0.75, 1.0, -2.0]          # 0.25/0.5 = 0.5 -> 0 (ties to even); 0.75/0.5 = 1.5 -> 2
    # row 0, group 1: all zero -> scale 0, codes 8
    # row 1, group 0: max 7 -> scale 1; row 1, group 1: max 14 -> scale 2
    x[1, 0], x[1, 1], x[1, 31] = 7.0, -3.0, 2.4
    x[1, 32], x[1, 33], x[1, 63] = -14.0, 5.0, 3.0                    # 5/2 = 2.5 -> 2 ; 3/2 = 1.5 -> 2
    b = synth.int4_g32_encode(x, H).reshape(2, H // 2 + 4)
    want0 = [7, -7, 1, -1, 0, 2, 2, -4] + [0] * 24
    codes0 = [(int(b[0, i // 2]) >> (4 * (i % 2))) & 15 for i in range(32)]
    assert codes0 == [q + 8 for q in want0]
    assert all(int(v) == 0x88 for v in b[0, 16:32])                   # the all-zero group: code 8 everywhere
    assert list(b[0, 32:36]) == [0x00, 0x3F, 0x00, 0x00]              # bf16(0.5) = 0x3F00, then bf16(0) little endian
    assert list(b[1, 32:36]) == [0x80, 0x3F, 0x00, 0x40]              # bf16(1.0) = 0x3F80, bf16(2.0) = 0x4000
    v = synth.int4_g32_decode(b.reshape(-1), H).reshape(2, H)
    assert list(v[0, :8]) == [3.5, -3.5, 0.5, -0.5, 0.0, 1.0, 1.0, -2.0] and not v[0, 8:].any()
    assert (v[1, 0], v[1, 1], v[1, 31], v[1, 32], v[1, 33], v[1, 63]) == (7.0, -3.0, 2.0, -14.0, 4.0, 4.0)
    # random rows: brute-force decode per element, error at most half a step of the group's stored scale,
    # the group maximum itself reproduced to the bf16 rounding of the scale
    rng = np.random.default_rng(1)
    H = 256
    y = (rng.standard_normal((5, H)) * 0.02).astype(np.float32)
    bb = synth.int4_g32_encode(y, H)
    assert bb.size == 5 * (H // 2 + 2 * (H // 32))
    dec = synth.int4_g32_decode(bb, H).reshape(5, H)
    rows = bb.reshape(5, -1)
    for r in range(5):
        for gidx in range(H // 32):
            sb = int(rows[r, H // 2 + 2 * gidx]) | (int(rows[r, H // 2 + 2 * gidx + 1]) << 8)
            scale = float(np.array([sb << 16], np.uint32).view(np.float32)[0])
            seg = y[r, 32 * gidx:32 * gidx + 32]
            assert abs(scale - np.abs(seg).max() / 7) <= 2.0 ** -8 * scale
            for j in range(32):
                byte = int(rows[r, (32 * gidx + j) // 2])
                code = (byte >> 4) if j % 2 else (byte & 15)
                assert 1 <= code <= 15
                val = (code - 8) * scale
                assert val == dec[r, 32 * gidx + j]
                assert abs(val - seg[j]) <= 0.5 * scale * (1 + 2.0 ** -7)
    shape = synth.Shape(1, 1024, 4, 2, 8, 0, 0, 0, 0, 3, 1)
    blk = synth.gen_expert_block(0, shape, 0, 1)
    assert blk.dtype == np.uint8 and blk.size == synth.expert_block_bytes(shape) == 3 * 8 * (512 + 64)
    assert synth.gen_router(0, shape, 0).dtype == np.uint16
    w = synth.widen(shape, blk)
    assert w.size == 3 * 8 * 1024 and 0.015 < w.std() < 0.025
