"""The give-up path of the bounded device-side waits, exercised without
hanging anything: with fb_tuning.wait_cycles = -1 every wait of the tcgen05
kernels gives up at once (no spinning), so the launch stops issuing work with
bulk copies still in flight, drains, frees its tensor memory, reports
FB_ST_DEV_TIMEOUT and returns.  What matters afterwards: the call came back,
the status bit is there, and the same context computes correct results again
-- on the same work list and on a fresh one."""
import numpy as np
import pytest
import torch

from oracle import flowblock_oracle as O
from paper_2607_17652_b200 import binding as B
from paper_2607_17652_b200 import synth
from tests import harness as H

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_attention_gives_up_reports_and_recovers():
    wl = synth.tiny_workload(prefix_lo=200, prefix_hi=900, n_requests=4)
    stc = synth.make_structure(wl)
    tokens = synth.make_tokens(stc)
    attn = synth.make_attn_inputs(stc)
    ctx = B.Context(**H.common_cfg(stc))
    st = B.DeviceState.from_numpy(DEV, stc.active, stc.prefix_len, stc.L, stc.R, tokens,
                                  np.zeros((wl.n_requests, wl.wmax), np.uint8), stc.page_table)
    pk = B.PackBuffers.alloc(ctx, DEV)
    sb = B.StepBuffers(ctx, DEV)
    q, kw, vw, kp, vp = (t.to(DEV) for t in attn)
    ocfg = H.oracle_cfg(stc)
    opk = O.pack_wavefronts(ocfg, H.oracle_state(stc, tokens))
    ref = O.wavefront_attn(ocfg, opk, *(H.f64(t) for t in attn), stc.page_table)
    rows = H.live_rows(opk, wl.block_len)

    B.fb_pack_wavefronts(ctx, st, pk, sb.ws, sb.status)
    ctx.set_tuning(wait_cycles=-1)                       # every wait gives up at once
    B.fb_wavefront_attn(ctx, pk, q, kw, vw, kp, vp, st.page_table, sb.out, sb.ws, sb.status)
    torch.cuda.synchronize()                             # the launch ended by itself
    assert int(sb.status.item()) & B.FB_ST_DEV_TIMEOUT
    assert int(sb.status.item()) & ~B.FB_ST_DEV_TIMEOUT == 0

    ctx.set_tuning()                                     # default limit again
    for fresh_pack in (False, True):
        # first on the work list the aborted launch had started to hand out, then on a new one
        sb.status.zero_()
        sb.out.fill_(7.0)
        if fresh_pack:
            B.fb_pack_wavefronts(ctx, st, pk, sb.ws, sb.status)
        B.fb_wavefront_attn(ctx, pk, q, kw, vw, kp, vp, st.page_table, sb.out, sb.ws, sb.status)
        torch.cuda.synchronize()
        assert int(sb.status.item()) == 0
        max_abs, rel = H.attn_errors(sb.out, ref, rows)
        assert max_abs <= 1e-2 and rel <= 5e-3, (fresh_pack, max_abs, rel)
        assert bool((sb.out[len(rows):].float() == 7.0).all())


def test_lm_head_gives_up_reports_and_recovers():
    wl = synth.tiny_workload()
    stc = synth.make_structure(wl)
    tokens = synth.make_tokens(stc)
    hidden = 128
    x, w, tokens = synth.make_lm_head_inputs(stc, tokens, hidden)
    ctx = B.Context(**H.common_cfg(stc))
    st = B.DeviceState.from_numpy(DEV, stc.active, stc.prefix_len, stc.L, stc.R, tokens,
                                  np.zeros((wl.n_requests, wl.wmax), np.uint8), stc.page_table)
    pk = B.PackBuffers.alloc(ctx, DEV)
    sb = B.StepBuffers(ctx, DEV)
    ws = torch.zeros(B.lib().fb_lm_head_workspace_bytes(ctx.handle), dtype=torch.uint8, device=DEV)
    dx, dw = x.to(DEV), w.to(DEV)
    B.fb_pack_wavefronts(ctx, st, pk, sb.ws, sb.status)
    tokens_dev = st.tokens.clone()
    ctx.set_tuning(wait_cycles=-1)
    B.fb_lm_head_t2t(ctx, pk, dx, dw, st, sb.argmax, sb.conf, sb.action, sb.slot_stats, ws, sb.status)
    torch.cuda.synchronize()
    assert int(sb.status.item()) & B.FB_ST_DEV_TIMEOUT
    ctx.set_tuning()
    st.tokens.copy_(tokens_dev)                          # outputs of the aborted call are undefined
    sb.status.zero_()
    B.fb_lm_head_t2t(ctx, pk, dx, dw, st, sb.argmax, sb.conf, sb.action, sb.slot_stats, ws, sb.status)
    torch.cuda.synchronize()
    assert int(sb.status.item()) == 0
    ocfg = H.oracle_cfg(stc)
    ost = H.oracle_state(stc, tokens)
    opk = O.pack_wavefronts(ocfg, ost)
    xhat, conf = O.lm_head_rows(ocfg, opk, H.f64(x), H.f64(w))
    np.testing.assert_array_equal(sb.argmax.cpu().numpy(), xhat)
    np.testing.assert_allclose(sb.conf.cpu().numpy(), conf, rtol=0, atol=5e-5)
    action, stats = O.t2t_update(ocfg, opk, ost, xhat, conf)
    np.testing.assert_array_equal(sb.action.cpu().numpy(), action)
    np.testing.assert_array_equal(st.tokens.cpu().numpy(), ost.tokens)
