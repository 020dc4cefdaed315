"""fb_wavefront_attn_static: the attention call for callers that may not
allocate device memory (an engine whose pool owns the whole device, a plugin
in a pre-partitioned process, a loop that must avoid cudaMalloc's implicit
synchronisation).  Its scratch is a fixed array inside the library, so the
call takes no workspace.  Checked here against the CPU oracle (its work list
never splits the key axis, a different schedule from the regular call's) and
against the regular entry point, twice in a row (the array keeps the first
call's contents), and against its size limit.  This file sorts last on purpose: a run that stops at the first failure
has then already run every other test."""
import numpy as np
import pytest
import torch

from oracle import flowblock_oracle as O
from paper_2607_17652_b200 import binding as B
from paper_2607_17652_b200 import synth
from tests import harness as H

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
ATTN_MAX_ABS, ATTN_REL_L2 = 1e-2, 5e-3     # the tolerance of the attention parity tests


def _setup(wl, seed=None):
    stc = synth.make_structure(wl, seed)
    tokens = synth.make_tokens(stc)
    attn = synth.make_attn_inputs(stc)
    ctx = B.Context(**synth.config_dict(stc))
    st = B.DeviceState.from_numpy(DEV, stc.active, stc.prefix_len, stc.L, stc.R, tokens,
                                  np.zeros((wl.n_requests, wl.wmax), np.uint8), stc.page_table)
    pk = B.PackBuffers.alloc(ctx, DEV)
    sb = B.StepBuffers(ctx, DEV)
    return stc, ctx, st, pk, sb, [t.to(DEV) for t in attn]


def _oracle_attn(stc, q, kw, vw, kp, vp):
    """fp64 attention of the oracle on the same bytes."""
    ocfg = H.oracle_cfg(stc)
    opk = O.pack_wavefronts(ocfg, H.oracle_state(stc, synth.make_tokens(stc)))
    ref = O.wavefront_attn(ocfg, opk, *(H.f64(t.cpu()) for t in (q, kw, vw, kp, vp)), stc.page_table)
    return ref, H.live_rows(opk, stc.wl.block_len)


@pytest.mark.parametrize("wl", [synth.tiny_workload(prefix_lo=300, prefix_hi=2500, n_requests=5),
                                synth.WORKLOADS[1]], ids=["tiny_long", "cfg1"])
def test_static_scratch_attention_matches_workspace_attention(wl):
    stc, ctx, st, pk, sb, (q, kw, vw, kp, vp) = _setup(wl)
    live = synth.n_live_slots(stc) * wl.block_len
    # reference: the regular entry points with a caller-allocated workspace
    B.fb_pack_wavefronts(ctx, st, pk, sb.ws, sb.status)
    B.fb_wavefront_attn(ctx, pk, q, kw, vw, kp, vp, st.page_table, sb.out, sb.ws, sb.status)
    torch.cuda.synchronize()
    want = sb.out[:live].float().clone()
    pack_ref = {k: v.copy() for k, v in pk.to_numpy().items()}
    ref, ref_rows = _oracle_attn(stc, q, kw, vw, kp, vp)
    assert len(ref_rows) == live
    for call in range(2):                       # two calls in a row share the array
        out = torch.full_like(sb.out, 3.0)
        B.fb_wavefront_attn_static(ctx, st, pk, q, kw, vw, kp, vp, out, sb.status)
        torch.cuda.synchronize()
        assert int(sb.status.item()) == 0
        o_abs, o_rel = H.attn_errors(out, ref, ref_rows)                # against the oracle
        assert o_abs <= ATTN_MAX_ABS and o_rel <= ATTN_REL_L2, (call, o_abs, o_rel)
        got = out[:live].float()                                        # and against the regular call
        max_abs = float((got - want).abs().max())
        rel = float((got - want).norm() / want.norm())
        assert max_abs <= ATTN_MAX_ABS and rel <= ATTN_REL_L2, (call, max_abs, rel)
        assert bool((out[live:].float() == 3.0).all())          # padding rows untouched
        for k, v in pk.to_numpy().items():                      # pack arrays rewritten identically
            np.testing.assert_array_equal(v, pack_ref[k], err_msg=k)
    # a different batch right after: nothing of the previous work list may leak
    stc2, ctx2, st2, pk2, sb2, (q2, kw2, vw2, kp2, vp2) = _setup(wl, seed=stc.seed + 77)
    live2 = synth.n_live_slots(stc2) * wl.block_len
    B.fb_pack_wavefronts(ctx2, st2, pk2, sb2.ws, sb2.status)
    B.fb_wavefront_attn(ctx2, pk2, q2, kw2, vw2, kp2, vp2, st2.page_table, sb2.out, sb2.ws, sb2.status)
    out2 = torch.zeros_like(sb2.out)
    B.fb_wavefront_attn_static(ctx2, st2, pk2, q2, kw2, vw2, kp2, vp2, out2, sb2.status)
    torch.cuda.synchronize()
    ref2, rows2 = _oracle_attn(stc2, q2, kw2, vw2, kp2, vp2)
    o_abs, o_rel = H.attn_errors(out2, ref2, rows2)
    assert o_abs <= ATTN_MAX_ABS and o_rel <= ATTN_REL_L2, (o_abs, o_rel)
    d = (out2[:live2].float() - sb2.out[:live2].float())
    assert float(d.abs().max()) <= ATTN_MAX_ABS
    assert float(d.norm() / sb2.out[:live2].float().norm()) <= ATTN_REL_L2


def test_static_scratch_rejects_configurations_beyond_its_size():
    big = dict(max_requests=16384, wmax=8, block_len=32, n_q_heads=32, n_kv_heads=8, head_dim=128,
               page_size=64, num_pages=16, max_pages_per_req=4, vocab=1024, mask_id=1023, eos_id=1022,
               max_blocks=8, s_pe=1, tau_mask=0.9, tau_edit=0.95, theta_spawn=0.5, sm_scale=0.0)
    ctx = B.Context(**big)
    dummy = torch.zeros(64, dtype=torch.int32, device=DEV)
    st = B.fb_state(*([dummy.data_ptr()] * 7))
    pk = B.fb_pack(*([dummy.data_ptr()] * 9))
    import ctypes as C
    rc = B.lib().fb_wavefront_attn_static(ctx.handle, C.byref(st), C.byref(pk), *([dummy.data_ptr()] * 7), None)
    assert rc == B.FB_ERR_WORKSPACE
    msg = B.lib().fb_last_error(ctx.handle).decode()
    assert "8 MiB" in msg and "fb_wavefront_attn" in msg
