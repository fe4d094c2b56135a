"""The allocation-free expert-sum entry point against the regular decode step.

Collected last on purpose: if it fails, a run that stops at the first failure has already
run everything else.  The entry point is for embedders that may not call cudaMalloc where
they use the library (device memory handed out once at start-up by another component,
allocator calls banned on worker threads, a device that is already full); it keeps its
scratch in a fixed device array inside the library instead.  Here the same layer is
evaluated by remoe_decode_step (scratch allocated at stack creation) and by
remoe_expert_ffn_static, twice in a row with different inputs, and the two outputs must
agree within the tolerance the parity tests use -- with each other and with the CPU oracle's
expert sum for the same ids and gate weights.  The second call must also leave the amount of
free device memory exactly as it found it.
"""
import numpy as np
import pytest

import synth

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("shape", [
    synth.Shape(1, 2048, 24, 6, 352, 2, 352, 0, 0, 1, 1),      # bf16, full width, shared experts
    synth.Shape(1, 256, 16, 2, 128, 0, 0, 0, 0, 0, 1),         # float32, the tiny configuration's shape
])
def test_static_entry_matches_decode_step_twice(shape):
    import torch
    from paper_2605_27081_b200 import binding as B
    from paper_2605_27081_b200.loader import LoadedWorkload
    from oracle import remoe_oracle as orc
    from parity_util import TOL, rel_err, widen

    wl = LoadedWorkload(shape, shape.n_routed, seed=11)
    try:
        H, K = shape.hidden, shape.top_k
        dev_blocks = [torch.from_numpy(wl.expert_block(0, e).copy()).to("cuda") for e in range(shape.n_routed)]
        dev_shared = [torch.from_numpy(b.copy()).to("cuda") for b in wl.shared[0]]
        d_in = torch.empty((1, 1, H), dtype=torch.float32, device="cuda")
        d_out = torch.empty_like(d_in)
        d_ids = torch.empty((1, 1, K), dtype=torch.int32, device="cuda")
        d_g = torch.empty((1, 1, K), dtype=torch.float32, device="cuda")
        out_static = torch.empty(H, dtype=torch.float32, device="cuda")
        hs = synth.HiddenStream(11, shape, 0.3)
        for call in range(2):
            d_in.copy_(torch.from_numpy(hs.step()))
            wl.stack.decode_step(d_in, d_out, d_ids, d_g)
            torch.cuda.synchronize()
            ids = d_ids.cpu().numpy().reshape(-1)
            gates = d_g.cpu().numpy().reshape(-1)
            blocks = [dev_blocks[int(e)] for e in ids] + dev_shared
            inter = [shape.inter_routed] * K + [shape.inter_shared] * shape.n_shared
            scales = [float(g) for g in gates] + [1.0] * shape.n_shared
            out_static.fill_(float("nan"))
            torch.cuda.synchronize()
            free_before = torch.cuda.mem_get_info()[0]
            rc = B.remoe_expert_ffn_static(H, shape.weight_dtype, blocks, inter, scales, d_in, out_static)
            assert rc == B.REMOE_OK
            torch.cuda.synchronize()
            if call == 1:
                # the first call on a device loads the kernels and looks up the scratch address; from
                # the second on a call must not change what the device has free
                assert torch.cuda.mem_get_info()[0] == free_before
            ref = d_out.cpu().numpy().reshape(-1)
            got = out_static.cpu().numpy()
            assert np.isfinite(got).all()
            assert rel_err(got, ref) <= TOL[shape.weight_dtype], (call, rel_err(got, ref))
            # and against the oracle's expert sum for the same ids and gate weights
            x = d_in.cpu().numpy().reshape(-1)
            o_ref = orc.moe_output(
                x, ids, gates, shape.n_routed,
                lambda e: synth.expert_matrices(widen(shape, wl.expert_block(0, e)), H, shape.inter_routed),
                [synth.expert_matrices(widen(shape, b), H, shape.inter_shared) for b in wl.shared[0]],
                mode="selected")
            assert rel_err(got, o_ref) <= TOL[shape.weight_dtype], (call, rel_err(got, o_ref))
        # one small expert: fewer rows than CTAs, so most CTAs own nothing; and an input that is also the output
        e0 = int(ids[0])
        one = orc.moe_output(x, [e0], [0.75], shape.n_routed,
                             lambda e: synth.expert_matrices(widen(shape, wl.expert_block(0, e)), H, shape.inter_routed),
                             mode="selected")
        few = 24                                            # rows of the block used: its first `few` channels
        w_g, w_u, w_d = synth.expert_matrices(widen(shape, wl.expert_block(0, e0)), H, shape.inter_routed)
        one_few = 0.75 * orc.swiglu_expert(w_g[:few], w_u[:few], w_d[:, :few], x)
        assert B.remoe_expert_ffn_static(H, shape.weight_dtype, [dev_blocks[e0]], [few], [0.75], d_in,
                                         out_static) == B.REMOE_OK
        torch.cuda.synchronize()
        assert rel_err(out_static.cpu().numpy(), one_few) <= TOL[shape.weight_dtype]
        inplace = d_in.reshape(-1).clone()
        assert B.remoe_expert_ffn_static(H, shape.weight_dtype, [dev_blocks[e0]], [shape.inter_routed], [0.75],
                                         inplace, inplace) == B.REMOE_OK
        torch.cuda.synchronize()
        assert rel_err(inplace.cpu().numpy(), one) <= TOL[shape.weight_dtype]
        # an element type the entry point has no kernel for
        assert B.remoe_expert_ffn_static(H, B.REMOE_FP8_E4M3, [dev_blocks[0]], [8], [1.0],
                                         d_in, out_static) == B.REMOE_E_UNSUPPORTED
        assert B.remoe_expert_ffn_static(H, 7, [dev_blocks[0]], [8], [1.0], d_in, out_static) == B.REMOE_E_ARG
        # sizes beyond the fixed scratch are refused before anything is launched
        too_many = [dev_blocks[0]] * 17
        assert B.remoe_expert_ffn_static(H, shape.weight_dtype, too_many, [shape.inter_routed] * 17, [1.0] * 17,
                                         d_in, out_static) == B.REMOE_E_UNSUPPORTED
        assert B.remoe_expert_ffn_static(4096, shape.weight_dtype, [dev_blocks[0]], [8], [1.0],
                                         d_in, out_static) == B.REMOE_E_UNSUPPORTED
        assert B.remoe_expert_ffn_static(H, shape.weight_dtype, [dev_blocks[0]], [1 << 20], [1.0],
                                         d_in, out_static) == B.REMOE_E_UNSUPPORTED
        assert B.remoe_expert_ffn_static(H, shape.weight_dtype, [dev_blocks[0]], [0], [1.0],
                                         d_in, out_static) == B.REMOE_E_ARG
    finally:
        wl.close()
