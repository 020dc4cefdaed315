"""The CTA-pair attention kernel (fb_tuning.attn_pair = 1: four Q tiles of one
request and KV head on a cluster of two CTAs that share every K/V tile, the
other tiles on single CTAs) against the oracle, at the tolerance of the
single-CTA kernel: shapes whose requests hold one or more quads plus leftovers,
forced key-axis splits, the window resident in the pages, scores that force the
softmax reference to move, and the give-up path of its bounded waits."""
import numpy as np
import pytest
import torch

from oracle import flowblock_oracle as O
from paper_2607_17652_b200 import binding as B
from paper_2607_17652_b200 import synth
from tests import harness as H

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
ATTN_MAX_ABS, ATTN_REL_L2 = 1e-2, 5e-3

SHAPES = {
    # one tile per slot, up to four live blocks: a quad only where W_r = 4
    "b32_w4": synth.tiny_workload(head_dim=128, n_q_heads=8, n_kv_heads=2, wmax=4, w_lo=1, w_hi=4, n_requests=6,
                                  prefix_lo=100, prefix_hi=900, max_blocks=16),
    # two tiles per slot, three live blocks: a quad and a pair per KV head
    "b64_w3": synth.tiny_workload(head_dim=128, n_q_heads=8, n_kv_heads=2, block_len=64, wmax=3, w_lo=2, w_hi=3,
                                  n_requests=4, prefix_lo=0, prefix_hi=700),
    # group of 8: two tiles per slot; four blocks: two quads per KV head, nothing left over
    "g8_w4": synth.tiny_workload(head_dim=128, n_q_heads=16, n_kv_heads=2, wmax=4, w_lo=4, w_hi=4, n_requests=3,
                                 prefix_lo=60, prefix_hi=420, max_blocks=16),
    # five blocks of 128 tokens, one head per group: five tiles per head, a quad and a leftover tile
    "mha_b128_w5": synth.tiny_workload(head_dim=128, n_q_heads=2, n_kv_heads=2, block_len=128, wmax=5, w_lo=3, w_hi=5,
                                       n_requests=3, prefix_lo=3, prefix_hi=260, max_blocks=16),
    "long": synth.tiny_workload(head_dim=128, n_q_heads=8, n_kv_heads=2, wmax=4, w_lo=3, w_hi=4, n_requests=3,
                                prefix_lo=3000, prefix_hi=6000, max_blocks=16),
}


def _run(wl, tuning, window_in_pages=0, attn=None, seed=None):
    stc = synth.make_structure(wl, seed)
    tokens = synth.make_tokens(stc)
    attn = synth.make_attn_inputs(stc) if attn is None else attn
    ctx = B.Context(tuning=dict(tuning, attn_pair=1), **H.common_cfg(stc, window_in_pages=window_in_pages))
    act = stc.active == 1
    plan = ctx.attn_plan(stc.prefix_len[act], (stc.R - stc.L)[act])
    assert plan["pair"]["items"] > 0, "no quad in this workload: the pair kernel would not run"
    st = B.DeviceState.from_numpy(DEV, stc.active, stc.prefix_len, stc.L, stc.R, tokens,
                                  np.zeros((wl.n_requests, wl.wmax), np.uint8), stc.page_table)
    pk = B.PackBuffers.alloc(ctx, DEV)
    sb = B.StepBuffers(ctx, DEV)
    q, kw, vw, kp, vp = (t.to(DEV) for t in attn)
    sb.out.fill_(7.0)
    B.fb_pack_wavefronts(ctx, st, pk, sb.ws, sb.status)
    if window_in_pages:
        B.fb_scatter_window_kv(ctx, pk, st.page_table, kw, vw, kp, vp, sb.status)
        B.fb_wavefront_attn(ctx, pk, q, None, None, kp, vp, st.page_table, sb.out, sb.ws, sb.status)
    else:
        B.fb_wavefront_attn(ctx, pk, q, kw, vw, kp, vp, st.page_table, sb.out, sb.ws, sb.status)
    torch.cuda.synchronize()
    assert int(sb.status.item()) == 0, int(sb.status.item())
    ocfg = H.oracle_cfg(stc)
    opk = O.pack_wavefronts(ocfg, H.oracle_state(stc, tokens))
    ref = O.wavefront_attn(ocfg, opk, *(H.f64(t) for t in attn), stc.page_table)
    rows = H.live_rows(opk, wl.block_len)
    max_abs, rel = H.attn_errors(sb.out, ref, rows)
    assert max_abs <= ATTN_MAX_ABS and rel <= ATTN_REL_L2, (max_abs, rel)
    assert bool((sb.out[len(rows):].float() == 7.0).all())
    return plan


@pytest.mark.parametrize("name", list(SHAPES))
@pytest.mark.parametrize("window_in_pages", [0, 1])
def test_pair_kernel_matches_oracle(name, window_in_pages):
    _run(SHAPES[name], {}, window_in_pages)


@pytest.mark.parametrize("target", [1, 40, 100000])
def test_pair_kernel_with_forced_key_axis_splits(target):
    plan = _run(SHAPES["long"], dict(attn_target_items=target))
    assert (plan["pair"]["parts"] > 0) == (target > 1)


@pytest.mark.parametrize("factor", [6.0, 40.0])
@pytest.mark.parametrize("where", ["second_tile", "window"])
def test_pair_kernel_when_the_softmax_reference_moves(where, factor):
    """Keys far larger than what earlier key tiles held (in the second prefix
    tile of every request, or in its window): the re-based reference, the
    rescaled output and the redone tile must agree with the plain softmax.  V is
    halved so that near-one-hot output rows round to bf16 within the tolerance."""
    wl = SHAPES["b32_w4"]
    stc = synth.make_structure(wl)
    q, kw, vw, kp, vp = synth.make_attn_inputs(stc)
    vw, vp = (vw.float() * 0.5).to(torch.bfloat16), (vp.float() * 0.5).to(torch.bfloat16)
    if where == "second_tile":
        for r in range(wl.n_requests):
            if stc.prefix_len[r] > 200:
                page = int(stc.page_table[r, 2])
                kp[page] = (kp[page].float() * factor).to(torch.bfloat16)
    else:
        kw = (kw.float() * factor).to(torch.bfloat16)
    _run(wl, {}, attn=(q, kw, vw, kp, vp))


def test_pair_kernel_gives_up_reports_and_recovers():
    wl = SHAPES["b64_w3"]
    stc = synth.make_structure(wl)
    tokens = synth.make_tokens(stc)
    attn = synth.make_attn_inputs(stc)
    ctx = B.Context(tuning=dict(attn_pair=1), **H.common_cfg(stc))
    st = B.DeviceState.from_numpy(DEV, stc.active, stc.prefix_len, stc.L, stc.R, tokens,
                                  np.zeros((wl.n_requests, wl.wmax), np.uint8), stc.page_table)
    pk = B.PackBuffers.alloc(ctx, DEV)
    sb = B.StepBuffers(ctx, DEV)
    q, kw, vw, kp, vp = (t.to(DEV) for t in attn)
    B.fb_pack_wavefronts(ctx, st, pk, sb.ws, sb.status)
    ctx.set_tuning(attn_pair=1, wait_cycles=-1)              # every wait of both kernels gives up at once
    B.fb_wavefront_attn(ctx, pk, q, kw, vw, kp, vp, st.page_table, sb.out, sb.ws, sb.status)
    torch.cuda.synchronize()
    assert int(sb.status.item()) == B.FB_ST_DEV_TIMEOUT
    ctx.set_tuning(attn_pair=1)
    sb.status.zero_()
    sb.out.fill_(7.0)
    B.fb_wavefront_attn(ctx, pk, q, kw, vw, kp, vp, st.page_table, sb.out, sb.ws, sb.status)   # same work lists
    torch.cuda.synchronize()
    assert int(sb.status.item()) == 0
    ocfg = H.oracle_cfg(stc)
    opk = O.pack_wavefronts(ocfg, H.oracle_state(stc, tokens))
    ref = O.wavefront_attn(ocfg, opk, *(H.f64(t) for t in attn), stc.page_table)
    max_abs, rel = H.attn_errors(sb.out, ref, H.live_rows(opk, wl.block_len))
    assert max_abs <= ATTN_MAX_ABS and rel <= ATTN_REL_L2, (max_abs, rel)
