"""GPU parity of the 8-bit (FP8 E4M3) KV pages against the oracle.

Stored bytes are integer work: fb_scatter_window_kv_fp8 must reproduce the
oracle's quantiser bit for bit (both round the binary32 quotient x / scale to
nearest even and saturate).  With the rotary embedding the kernel rotates in
fp32 and the oracle in fp64, so a value that lands within rounding distance of
a tie may fall to the neighbouring code: at most one code step, on a small
fraction of the elements.

fb_wavefront_attn_fp8 against wavefront_attn_fp8 (fp64 attention on the values
the pages hold, queries as given).  Tolerance, derived from the format and not
tuned: the kernel rounds Q and the softmax weights P to E4M3 (3 mantissa
bits).  Round-to-nearest leaves an error uniform in +-half a step; relative to
a value with mantissa m in [1, 2) that is (2^-4 / sqrt 3) / m, and over
log-uniform mantissas its rms is 0.7355 * 2^-4 / sqrt 3 = 2.65e-2.  A weight
therefore carries 2.65e-2 from its own rounding and, through the score
s = scale * sum_d q_d k_d with independent errors on the q_d, another
2.65e-2 * rms(q) * rms(k) = 2.65e-2 for N(0,1) queries and keys: 3.75e-2 per
weight in all, independent across keys.  With values independent of the
weights the output row inherits the same relative error, so rel-L2 is expected
at 3.75e-2; the bound is 1.5 x that.  Element-wise the error of a row has
standard deviation 3.75e-2 * sqrt(sum w_i^2) * rms(v) (rms(v) = 1 here); the
oracle gives sum w_i^2 per row, and with up to 10^6 elements compared the
bound is 6 of those standard deviations plus the 1e-2 of the bf16 output.
Cases in which both roundings are exact (zero queries; one key
that dominates) must meet the bf16 path's tolerance instead, which pins the key
set, the paging, the scales and the normalisation tightly."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import flowblock_oracle as O
from paper_2607_17652_b200 import binding as B
from paper_2607_17652_b200 import synth
from tests import harness as H

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
F8_EPS_W = 3.75e-2
F8_REL_L2 = 1.5 * F8_EPS_W
EXACT_MAX_ABS, EXACT_REL_L2 = 1e-2, 5e-3

SHAPES = {
    "g4_b32": synth.tiny_workload(head_dim=128, n_q_heads=8, n_kv_heads=2, prefix_lo=0, prefix_hi=700, n_requests=4),
    "g4_b64": synth.tiny_workload(head_dim=128, n_q_heads=8, n_kv_heads=2, block_len=64, prefix_lo=40, prefix_hi=900,
                                  n_requests=4),
    "g8_b32": synth.tiny_workload(head_dim=128, n_q_heads=16, n_kv_heads=2, prefix_lo=60, prefix_hi=420, n_requests=4),
    "mha_b128": synth.tiny_workload(head_dim=128, n_q_heads=2, n_kv_heads=2, block_len=128, wmax=2, w_lo=1, w_hi=2,
                                    prefix_lo=3, prefix_hi=300, n_requests=3, max_blocks=6),
    "long": synth.tiny_workload(head_dim=128, n_q_heads=8, n_kv_heads=2, prefix_lo=3000, prefix_hi=6000, n_requests=3,
                                wmax=4, w_lo=2, w_hi=4, max_blocks=16),
}


def _setup(wl, tuning=None, seed=None):
    stc = synth.make_structure(wl, seed)
    tokens = synth.make_tokens(stc)
    q, kw, vw, _, _ = synth.make_attn_inputs(stc)
    k8, v8, ks, vs = synth.make_fp8_kv(stc)
    ctx = B.Context(tuning=tuning, kv_fp8=1, **H.common_cfg(stc, window_in_pages=1))
    st = B.DeviceState.from_numpy(DEV, stc.active, stc.prefix_len, stc.L, stc.R, tokens,
                                  np.zeros((wl.n_requests, wl.wmax), np.uint8), stc.page_table)
    pk = B.PackBuffers.alloc(ctx, DEV)
    sb = B.StepBuffers(ctx, DEV)
    ocfg = H.oracle_cfg(stc)
    opk = O.pack_wavefronts(ocfg, H.oracle_state(stc, tokens))
    return dict(wl=wl, stc=stc, ctx=ctx, st=st, pk=pk, sb=sb, ocfg=ocfg, opk=opk,
                q=q, kw=kw, vw=vw, k8=k8, v8=v8, ks=ks, vs=vs)


def _run(c, q=None, k8=None, v8=None, scatter=True):
    """scatter (the quantiser) + attention on the GPU and in the oracle; returns (out, ref, live rows)."""
    ctx, st, pk, sb = c["ctx"], c["st"], c["pk"], c["sb"]
    q = c["q"] if q is None else q
    k8 = (c["k8"] if k8 is None else k8).clone()
    v8 = (c["v8"] if v8 is None else v8).clone()
    dk8, dv8, dks, dvs = k8.to(DEV), v8.to(DEV), c["ks"].to(DEV), c["vs"].to(DEV)
    sb.out.fill_(7.0)
    B.fb_pack_wavefronts(ctx, st, pk, sb.ws, sb.status)
    if scatter:
        B.fb_scatter_window_kv_fp8(ctx, pk, st.page_table, c["kw"].to(DEV), c["vw"].to(DEV), dk8, dv8, dks, dvs,
                                   sb.status)
    B.fb_wavefront_attn_fp8(ctx, pk, q.to(DEV), dk8, dv8, dks, dvs, st.page_table, sb.out, sb.ws, sb.status)
    torch.cuda.synchronize()
    assert int(sb.status.item()) == 0, int(sb.status.item())
    ok8, ov8 = k8.numpy().copy(), v8.numpy().copy()
    if scatter:
        O.scatter_window_kv_fp8(c["ocfg"], c["opk"], H.f64(c["kw"]), H.f64(c["vw"]), ok8, ov8, c["ks"].numpy(),
                                c["vs"].numpy(), c["stc"].page_table)
        np.testing.assert_array_equal(dk8.cpu().numpy(), ok8)      # the stored bytes, bit for bit
        np.testing.assert_array_equal(dv8.cpu().numpy(), ov8)
    ref = O.wavefront_attn_fp8(c["ocfg"], c["opk"], H.f64(q), ok8, ov8, c["ks"].numpy(), c["vs"].numpy(),
                               c["stc"].page_table)
    rows = H.live_rows(c["opk"], c["wl"].block_len)
    assert bool((sb.out[len(rows):].float() == 7.0).all())           # rows of padding slots are not written
    c["pools_f64"] = (O.e4m3_decode(ok8) * c["ks"].numpy()[None, :, None, None], H.f64(q))
    return sb.out, ref, rows


def _within_f8_bound(c, out, ref, rows):
    """rel-L2 of all live rows and the row-scaled element-wise bound of the module docstring."""
    kd, q64 = c["pools_f64"]
    n2 = O.wavefront_attn_weight_norms(c["ocfg"], c["opk"], q64, None, kd, c["stc"].page_table)
    g = out.float().cpu().numpy().astype(np.float64)[rows]
    err = np.abs(g - ref[rows])
    allowed = 6.0 * F8_EPS_W * np.sqrt(n2[rows])[:, :, None] + 1e-2
    rel = float(np.linalg.norm(g - ref[rows]) / np.linalg.norm(ref[rows]))
    worst = float((err / allowed).max())
    return rel, worst


@pytest.mark.parametrize("name", list(SHAPES))
def test_scatter_bytes_bit_exact_and_attention_within_the_derived_bound(name):
    c = _setup(SHAPES[name])
    out, ref, rows = _run(c)
    rel, worst = _within_f8_bound(c, out, ref, rows)
    assert rel <= F8_REL_L2 and worst <= 1.0, (rel, worst)
    assert rel >= 2e-3, "an error this small means the 8-bit products did not run"


@pytest.mark.parametrize("target", [1, 100000])
def test_split_kv_changes_nothing_beyond_rounding(target):
    c = _setup(SHAPES["long"], tuning=dict(attn_target_items=target))
    out, ref, rows = _run(c)
    rel, worst = _within_f8_bound(c, out, ref, rows)
    assert rel <= F8_REL_L2 and worst <= 1.0, (target, rel, worst)
    hdr = c["sb"].ws[:64].cpu().numpy().view(np.int32)
    assert (hdr[3] > 0) == (target > 1)


@pytest.mark.parametrize("name", ["g4_b32", "g8_b32", "long"])
def test_zero_queries_average_exactly_the_visible_values(name):
    """q = 0: every weight is the same power of two and the queries are zeros,
    so nothing is rounded in 8 bits: the output is the mean of the visible V
    values as the pages hold them (times the head's scale), at the bf16 path's
    tolerance.  Counts exactly o_r + (s+1) bl keys per row, through the pages."""
    c = _setup(SHAPES[name])
    out, ref, rows = _run(c, q=torch.zeros_like(c["q"]))
    max_abs, rel = H.attn_errors(out, ref, rows)
    assert max_abs <= EXACT_MAX_ABS and rel <= EXACT_REL_L2, (max_abs, rel)


def test_one_dominant_key_returns_its_value():
    """A key whose score leads all others by far takes weight 1 (exact in 8
    bits), the output row is that key's value row."""
    wl = SHAPES["g4_b32"]
    c = _setup(wl)
    stc, opk = c["stc"], c["opk"]
    k8 = c["k8"].clone()
    q = c["q"].clone()
    ks = c["ks"].numpy()
    # for every request: key position 7 of its prefix (if it has one) gets +-448 codes along the
    # sign of a fixed direction, and every query of the request points that way
    direction = torch.sign(synth.randn_bf16((wl.head_dim,), stc.seed, 21).float())
    big = torch.where(direction > 0, torch.tensor(0x7E), torch.tensor(0xFE)).to(torch.uint8)   # +-448
    picked = {}
    for r in range(wl.n_requests):
        if stc.active[r] != 1 or stc.prefix_len[r] < 8:
            continue
        page = int(stc.page_table[r, 0])
        k8[page, :, 7, :] = big
        picked[r] = page
    for slot in range(opk.n_live):
        r = int(opk.slot_req[slot])
        if r in picked:
            q[slot * wl.block_len:(slot + 1) * wl.block_len] = (direction * 0.5).to(torch.bfloat16)
    out, ref, rows = _run(c, q=q, k8=k8, scatter=False)
    sel = np.concatenate([np.arange(s * wl.block_len, (s + 1) * wl.block_len) for s in range(opk.n_live)
                          if int(opk.slot_req[s]) in picked])
    assert len(sel) > 0
    max_abs, rel = H.attn_errors(out, ref, sel)
    assert max_abs <= EXACT_MAX_ABS and rel <= EXACT_REL_L2, (max_abs, rel)
    # and the oracle's rows are indeed the value row of that key
    v = O.e4m3_decode(c["v8"].numpy()) * c["vs"].numpy()[None, :, None, None]
    G = wl.n_q_heads // wl.n_kv_heads
    for s in range(opk.n_live):
        r = int(opk.slot_req[s])
        if r in picked:
            want = np.repeat(v[picked[r], :, 7, :], G, axis=0)
            assert np.abs(ref[s * wl.block_len] - want).max() < 1e-6


def test_constant_values_show_the_weight_rounding_is_unbiased():
    """V constant per head: the output is that constant times sum(rounded
    weights) / sum(weights).  Each row's ratio stays within the rounding error
    of a few dozen independent weights, and over all rows it averages to one:
    the E4M3 rounding of P carries no systematic bias into the output."""
    wl = SHAPES["long"]
    c = _setup(wl)
    v8 = torch.full_like(c["v8"], 0x3C)                     # 1.5 everywhere
    vw = torch.full_like(c["vw"], 1.5)
    c = dict(c, vw=vw)
    out, ref, rows = _run(c, v8=v8)
    G = wl.n_q_heads // wl.n_kv_heads
    got = out[:len(rows)].float().cpu().numpy().astype(np.float64)
    ratio = got / ref[:len(rows)]
    assert np.abs(ratio - 1).max() <= 3e-2, np.abs(ratio - 1).max()
    assert abs(ratio.mean() - 1) <= 3e-3, ratio.mean()


def test_rope_then_quantise_lands_on_the_oracle_code_or_its_neighbour():
    wl = SHAPES["g4_b32"]
    c = _setup(wl)
    ctx, st, pk, sb = c["ctx"], c["st"], c["pk"], c["sb"]
    dk8, dv8 = c["k8"].to(DEV), c["v8"].to(DEV)
    B.fb_pack_wavefronts(ctx, st, pk, sb.ws, sb.status)
    B.fb_scatter_window_kv_fp8(ctx, pk, st.page_table, c["kw"].to(DEV), c["vw"].to(DEV), dk8, dv8,
                               c["ks"].to(DEV), c["vs"].to(DEV), sb.status, rope_base=10000.0)
    torch.cuda.synchronize()
    assert int(sb.status.item()) == 0
    ok8, ov8 = c["k8"].numpy().copy(), c["v8"].numpy().copy()
    O.scatter_window_kv_fp8(c["ocfg"], c["opk"], H.f64(c["kw"]), H.f64(c["vw"]), ok8, ov8, c["ks"].numpy(),
                            c["vs"].numpy(), c["stc"].page_table, rope_base=10000.0)
    np.testing.assert_array_equal(dv8.cpu().numpy(), ov8)             # V is never rotated
    g = dk8.cpu().numpy()
    diff = g != ok8
    assert diff.mean() < 5e-3, diff.mean()
    # where they differ: neighbouring codes (the magnitude ordering of E4M3 codes is the integer
    # ordering of their low 7 bits)
    a, b = g[diff].astype(np.int32), ok8[diff].astype(np.int32)
    same_sign = (a & 0x80) == (b & 0x80)
    step = np.where(same_sign, np.abs((a & 0x7F) - (b & 0x7F)), (a & 0x7F) + (b & 0x7F))
    assert (step <= 1).all()


def test_contexts_that_cannot_hold_8_bit_pages_are_refused():
    wl = synth.tiny_workload()                                  # head_dim 64, window in slot order
    stc = synth.make_structure(wl)
    for over in (dict(), dict(window_in_pages=1)):
        ctx = B.Context(**H.common_cfg(stc, **over))
        pk = B.PackBuffers.alloc(ctx, DEV)
        d = torch.zeros(64, dtype=torch.float32, device=DEV)
        with pytest.raises(B.FlowBlockError) as e:
            B.fb_wavefront_attn_fp8(ctx, pk, d, d, d, d, d, d, d, d, d)
        assert e.value.code == B.FB_ERR_UNSUPPORTED


def test_multi_step_trajectory_with_8_bit_pages():
    """Eight consecutive steps with the pages in 8 bits: pack -> scatter (the
    quantiser, Eq. 6 every step) -> attention over the pages -> T2T ->
    gate/commit as a pointer bump.  After every step the pools must hold exactly
    the oracle's bytes (so the K/V of every block that retires is frozen as it
    was quantised in its last step, and nothing else moves), the state and the
    decisions must be bit-exact, the attention within the derived bound."""
    wl = synth.tiny_workload(head_dim=128, n_q_heads=8, n_kv_heads=2, n_requests=5, wmax=3, w_lo=1, w_hi=2,
                             prefix_lo=40, prefix_hi=400, max_blocks=10)
    stc = synth.make_structure(wl, n_inactive=2)
    late = [int(r) for r in np.flatnonzero(stc.active == 0)]
    tokens = synth.make_tokens(stc)
    ctx = B.Context(kv_fp8=1, **H.common_cfg(stc, window_in_pages=1, s_pe=1))
    st = B.DeviceState.from_numpy(DEV, stc.active, stc.prefix_len, stc.L, stc.R, tokens,
                                  np.zeros((wl.n_requests, wl.wmax), np.uint8), stc.page_table)
    pk = B.PackBuffers.alloc(ctx, DEV)
    sb = B.StepBuffers(ctx, DEV)
    ocfg = H.oracle_cfg(stc, s_pe=1)
    ost = H.oracle_state(stc, tokens)
    q, kw, vw, _, _ = synth.make_attn_inputs(stc)
    k8, v8, ks, vs = synth.make_fp8_kv(stc)
    ok8, ov8 = k8.numpy().copy(), v8.numpy().copy()
    dk8, dv8, dks, dvs = k8.to(DEV), v8.to(DEV), ks.to(DEV), vs.to(DEV)
    total_commits = 0
    for step in range(8):
        if step in (2, 4):
            r = late[step // 2 - 1]
            ost.active[r] = 1
            st.active[r] = 1
        cur = dataclasses.replace(stc)
        cur.active, cur.prefix_len, cur.L, cur.R = (ost.active.copy(), ost.prefix_len.copy(),
                                                   ost.L.copy(), ost.R.copy())
        z, tok2 = synth.make_logits(cur, ost.tokens, "calibrated", seed_shift=step, conf_shift=0.05 * step)
        ost.tokens[:] = tok2
        st.tokens.copy_(torch.from_numpy(tok2))
        q = synth.randn_bf16(q.shape, stc.seed + step, 1)
        kw = synth.randn_bf16(kw.shape, stc.seed + step, 2)
        vw = synth.randn_bf16(vw.shape, stc.seed + step, 3)
        B.fb_pack_wavefronts(ctx, st, pk, sb.ws, sb.status)
        B.fb_scatter_window_kv_fp8(ctx, pk, st.page_table, kw.to(DEV), vw.to(DEV), dk8, dv8, dks, dvs, sb.status)
        B.fb_wavefront_attn_fp8(ctx, pk, q.to(DEV), dk8, dv8, dks, dvs, st.page_table, sb.out, sb.ws, sb.status)
        B.fb_t2t_step(ctx, pk, z.to(DEV), st, sb.argmax, sb.conf, sb.action, sb.slot_stats, sb.status)
        B.fb_gate_commit(ctx, pk, sb.slot_stats, st, None, None, None, None, sb.n_committed, sb.spawned,
                         sb.step_counters, sb.status)
        torch.cuda.synchronize()
        assert int(sb.status.item()) == 0
        opk = O.pack_wavefronts(ocfg, ost)
        O.scatter_window_kv_fp8(ocfg, opk, H.f64(kw), H.f64(vw), ok8, ov8, ks.numpy(), vs.numpy(), ost.page_table)
        ref = O.wavefront_attn_fp8(ocfg, opk, H.f64(q), ok8, ov8, ks.numpy(), vs.numpy(), ost.page_table)
        rows = H.live_rows(opk, wl.block_len)
        g_out = sb.out.float().cpu().numpy().astype(np.float64)[rows]
        rel = float(np.linalg.norm(g_out - ref[rows]) / np.linalg.norm(ref[rows]))
        assert rel <= F8_REL_L2, (step, rel)
        xhat, conf = O.t2t_rows(ocfg, opk, H.f64(z))
        action, stats = O.t2t_update(ocfg, opk, ost, xhat, conf)
        ncom, spawned, ctr = O.gate_commit(ocfg, opk, stats, ost)          # window in the pages: nothing to copy
        np.testing.assert_array_equal(sb.action.cpu().numpy(), action)
        np.testing.assert_array_equal(sb.n_committed.cpu().numpy(), ncom)
        np.testing.assert_array_equal(sb.spawned.cpu().numpy(), spawned)
        np.testing.assert_array_equal(sb.step_counters.cpu().numpy(), ctr)
        g = st.to_numpy()
        for name in ("active", "prefix_len", "L", "R", "tokens", "pe_done"):
            np.testing.assert_array_equal(g[name], getattr(ost, name), err_msg=f"{name}@{step}")
        np.testing.assert_array_equal(dk8.cpu().numpy(), ok8, err_msg=f"K bytes@{step}")
        np.testing.assert_array_equal(dv8.cpu().numpy(), ov8, err_msg=f"V bytes@{step}")
        total_commits += int(ncom.sum())
    assert total_commits >= 3, "the trajectory never committed a block"
