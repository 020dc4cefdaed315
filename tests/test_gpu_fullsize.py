"""Parity at the benchmark's full size (64 heterogeneous requests, prefixes
1K-8K, V = 151,552), in the launch configuration bench.py times.  The oracle
cannot do the whole batch in seconds, so it recomputes sampled requests (all
their slots, rows and heads; every logits row of those slots) one by one, and
the rest is covered by properties that hold at any size."""
import numpy as np
import pytest
import torch

from oracle import flowblock_oracle as O
from paper_2607_17652_b200 import binding as B
from paper_2607_17652_b200 import synth
from tests import harness as H

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def full():
    wl = synth.WORKLOADS[2]
    stc = synth.make_structure(wl)
    tokens = synth.make_tokens(stc)
    n_live = synth.n_live_slots(stc)
    z_live, tokens = synth.make_logits(stc, tokens, "calibrated", n_rows=n_live * wl.block_len)
    attn = synth.make_attn_inputs(stc)
    ctx = B.Context(**synth.config_dict(stc))
    st = B.DeviceState.from_numpy(DEV, stc.active, stc.prefix_len, stc.L, stc.R, tokens,
                                  np.zeros((wl.n_requests, wl.wmax), np.uint8), stc.page_table)
    pk = B.PackBuffers.alloc(ctx, DEV)
    sb = B.StepBuffers(ctx, DEV)
    rows = ctx.max_slots * wl.block_len
    logits = torch.zeros(rows, wl.vocab, dtype=torch.bfloat16, device=DEV)
    logits[:z_live.shape[0]].copy_(z_live)
    q, kw, vw, kp, vp = (t.to(DEV) for t in attn)
    sb.out.fill_(7.0)
    B.fb_pack_wavefronts(ctx, st, pk, sb.ws, sb.status)
    B.fb_wavefront_attn(ctx, pk, q, kw, vw, kp, vp, st.page_table, sb.out, sb.ws, sb.status)
    B.fb_t2t_step(ctx, pk, logits, st, sb.argmax, sb.conf, sb.action, sb.slot_stats, sb.status)
    torch.cuda.synchronize()
    tokens_after = st.tokens.cpu().numpy().copy()
    kp_before = kp[:64].clone()
    B.fb_gate_commit(ctx, pk, sb.slot_stats, st, kw, vw, kp, vp, sb.n_committed, sb.spawned,
                     sb.step_counters, sb.status)
    torch.cuda.synchronize()
    assert int(sb.status.item()) == 0
    # requests to recompute: the longest and the shortest prefix, the widest window, a few more
    order = np.argsort(stc.prefix_len)
    keep = sorted({int(order[0]), int(order[-1]), int(np.argmax(stc.R - stc.L)), 5, 23, 41})
    return dict(wl=wl, stc=stc, tokens=tokens, tokens_after=tokens_after, attn=attn, z_live=z_live,
                ctx=ctx, st=st, pk=pk, sb=sb, keep=keep, n_live=n_live, logits=logits)


def test_pack_full_size_bit_exact(full):
    ref = O.pack_wavefronts(H.oracle_cfg(full["stc"]), H.oracle_state(full["stc"], full["tokens"]))
    g = full["pk"].to_numpy()
    assert int(g["n_live"][0]) == ref.n_live == full["n_live"]
    for name in ("slot_req", "slot_s", "slot_pos0", "slot_kv_len", "slot_flags", "req_slot_begin", "qtok", "pos"):
        np.testing.assert_array_equal(g[name], getattr(ref, name), err_msg=name)


def test_attention_sampled_requests(full):
    sp = H.sub_problem(full["stc"], full["tokens"], full["attn"], None, full["keep"])
    opk = O.pack_wavefronts(sp["ocfg"], sp["ost"])
    ref = O.wavefront_attn(sp["ocfg"], opk, sp["q"], sp["k_win"], sp["v_win"], sp["k_pool"], sp["v_pool"],
                           sp["ost"].page_table)
    n = len(sp["rows"])
    got = full["sb"].out[torch.from_numpy(sp["rows"]).to(DEV)].float().cpu().numpy().astype(np.float64)
    err = np.abs(got - ref[:n])
    rel = np.linalg.norm(got - ref[:n]) / np.linalg.norm(ref[:n])
    assert err.max() <= 1e-2 and rel <= 5e-3, (err.max(), rel)
    assert n >= 6 * 32


def test_attention_properties_all_rows(full):
    """Every live output row is a convex combination of V rows drawn from
    N(0,1): finite, and (softmax weights sum to one) bounded by the largest
    |v|; padding rows are untouched."""
    wl, sb, attn = full["wl"], full["sb"], full["attn"]
    live = full["n_live"] * wl.block_len
    out = sb.out[:live].float()
    assert bool(torch.isfinite(out).all())
    vmax = max(float(attn[2].float().abs().max()), float(attn[4].float().abs().max()))
    assert float(out.abs().max()) <= vmax + 1e-2
    assert bool((sb.out[live:].float() == 7.0).all())


def test_t2t_sampled_requests_and_global_properties(full):
    wl, stc, sb = full["wl"], full["stc"], full["sb"]
    sp = H.sub_problem(stc, full["tokens"], None, full["z_live"], full["keep"])
    opk = O.pack_wavefronts(sp["ocfg"], sp["ost"])
    xhat, conf = O.t2t_rows(sp["ocfg"], opk, sp["logits"])
    n = len(sp["rows"])
    for thr in (np.float32(wl.tau_mask), np.float32(wl.tau_edit)):
        assert np.abs(conf[:n] - float(thr)).min() >= 1e-3
    action, stats = O.t2t_update(sp["ocfg"], opk, sp["ost"], xhat, conf)
    rows = torch.from_numpy(sp["rows"]).to(DEV)
    np.testing.assert_array_equal(sb.argmax[rows].cpu().numpy(), xhat[:n])
    np.testing.assert_allclose(sb.conf[rows].cpu().numpy(), conf[:n], rtol=0, atol=2e-5)
    np.testing.assert_array_equal(sb.action[rows].cpu().numpy(), action[:n])
    for r in full["keep"]:
        np.testing.assert_array_equal(full["tokens_after"][r], sp["ost"].tokens[r], err_msg=f"tokens of request {r}")
    # properties over all live rows: the top-1 logit really is the row maximum,
    # the first index attaining it; confidences are probabilities
    live = full["n_live"] * wl.block_len
    z = full["logits"][:live]
    am = sb.argmax[:live].long()
    top = z.gather(1, am[:, None])[:, 0]
    assert bool((top == z.max(dim=1).values).all())
    first = (z == top[:, None]).float().argmax(dim=1)
    assert bool((first == am).all())
    cf = sb.conf[:live]
    assert bool(((cf > 0) & (cf <= 1.0)).all())
    # slot statistics are consistent with the per-position action codes
    act = sb.action[:live].view(full["n_live"], wl.block_len)
    st = sb.slot_stats[:full["n_live"]]
    assert bool(((act == 1).sum(1) == st[:, 2]).all()) and bool(((act == 2).sum(1) == st[:, 3]).all())
    assert int(sb.slot_stats[full["n_live"]:].abs().sum()) == 0


def test_gate_commit_sampled_requests(full):
    stc, sb = full["stc"], full["sb"]
    sp = H.sub_problem(stc, full["tokens"], full["attn"], full["z_live"], full["keep"])
    opk = O.pack_wavefronts(sp["ocfg"], sp["ost"])
    xhat, conf = O.t2t_rows(sp["ocfg"], opk, sp["logits"])
    action, stats = O.t2t_update(sp["ocfg"], opk, sp["ost"], xhat, conf)
    ncom, spawned, ctr = O.gate_commit(sp["ocfg"], opk, stats, sp["ost"], sp["k_win"], sp["v_win"],
                                       sp["k_pool"], sp["v_pool"])
    g = full["st"].to_numpy()
    for r in full["keep"]:
        assert int(sb.n_committed[r]) == int(ncom[r]) and int(sb.spawned[r]) == int(spawned[r])
        for name in ("active", "prefix_len", "L", "R"):
            assert int(g[name][r]) == int(getattr(sp["ost"], name)[r]), (name, r)
        np.testing.assert_array_equal(g["pe_done"][r], sp["ost"].pe_done[r])
        np.testing.assert_array_equal(g["tokens"][r], sp["ost"].tokens[r])
    # counters add up over the whole batch
    c = sb.step_counters.cpu().numpy()
    assert c[O.CT_BLOCKS] == int(sb.n_committed.sum()) and c[O.CT_SPAWNED] == int(sb.spawned.sum())
    assert c[O.CT_LIVE_SLOTS] == full["n_live"]


@pytest.fixture(scope="module")
def longctx():
    """The long-context workload (16 requests, prefixes of 16K-32K tokens, three
    live blocks of 64 tokens each) at full size, one whole step: pack,
    attention, the T2T step over V = 151,552 calibrated logits, gate/commit."""
    wl = synth.WORKLOADS[3]
    stc = synth.make_structure(wl)
    tokens = synth.make_tokens(stc)
    n_live = synth.n_live_slots(stc)
    z_live, tokens = synth.make_logits(stc, tokens, "calibrated", conf_shift=0.2, n_rows=n_live * wl.block_len)
    attn = synth.make_attn_inputs(stc)
    ctx = B.Context(**synth.config_dict(stc))
    st = B.DeviceState.from_numpy(DEV, stc.active, stc.prefix_len, stc.L, stc.R, tokens,
                                  np.zeros((wl.n_requests, wl.wmax), np.uint8), stc.page_table)
    pk = B.PackBuffers.alloc(ctx, DEV)
    sb = B.StepBuffers(ctx, DEV)
    logits = torch.zeros(ctx.max_slots * wl.block_len, wl.vocab, dtype=torch.bfloat16, device=DEV)
    logits[:z_live.shape[0]].copy_(z_live)
    q, kw, vw, kp, vp = (t.to(DEV) for t in attn)
    sb.out.fill_(7.0)
    B.fb_pack_wavefronts(ctx, st, pk, sb.ws, sb.status)
    B.fb_wavefront_attn(ctx, pk, q, kw, vw, kp, vp, st.page_table, sb.out, sb.ws, sb.status)
    B.fb_t2t_step(ctx, pk, logits, st, sb.argmax, sb.conf, sb.action, sb.slot_stats, sb.status)
    B.fb_gate_commit(ctx, pk, sb.slot_stats, st, kw, vw, kp, vp, sb.n_committed, sb.spawned,
                     sb.step_counters, sb.status)
    torch.cuda.synchronize()
    assert int(sb.status.item()) == 0
    return dict(wl=wl, stc=stc, tokens=tokens, attn=attn, z_live=z_live, st=st, sb=sb, n_live=n_live,
                keep=[0, wl.n_requests - 1])


def test_long_context_attention_sampled_requests(longctx):
    """The first request runs as whole work items, the last one falls into the
    stretch that the scheduler cuts into filler pieces (partial results +
    combine kernel); all slots of both against the oracle."""
    wl, stc, sb = longctx["wl"], longctx["stc"], longctx["sb"]
    hdr = sb.ws[:64].cpu().numpy().view(np.int32)
    assert hdr[3] > 0, "no unit was split: the filler path is not exercised"
    sp = H.sub_problem(stc, longctx["tokens"], longctx["attn"], None, longctx["keep"])
    opk = O.pack_wavefronts(sp["ocfg"], sp["ost"])
    ref = O.wavefront_attn(sp["ocfg"], opk, sp["q"], sp["k_win"], sp["v_win"], sp["k_pool"], sp["v_pool"],
                           sp["ost"].page_table)
    n = len(sp["rows"])
    got = sb.out[torch.from_numpy(sp["rows"]).to(DEV)].float().cpu().numpy().astype(np.float64)
    err = np.abs(got - ref[:n])
    rel = np.linalg.norm(got - ref[:n]) / np.linalg.norm(ref[:n])
    assert err.max() <= 1e-2 and rel <= 5e-3, (err.max(), rel)
    assert n == 2 * 3 * wl.block_len
    live = longctx["n_live"] * wl.block_len
    assert bool(torch.isfinite(sb.out[:live].float()).all())
    assert bool((sb.out[live:].float() == 7.0).all())


def test_long_context_t2t_and_gate_sampled_requests(longctx):
    """Eq. 1, the block counts, retirement and admission at the long-context
    shape (bl 64, W 3, 3072 rows of 151,552 logits): every row of the two
    sampled requests against the oracle's row pass, update and gate/commit."""
    wl, stc, sb = longctx["wl"], longctx["stc"], longctx["sb"]
    sp = H.sub_problem(stc, longctx["tokens"], longctx["attn"], longctx["z_live"], longctx["keep"])
    opk = O.pack_wavefronts(sp["ocfg"], sp["ost"])
    xhat, conf = O.t2t_rows(sp["ocfg"], opk, sp["logits"])
    n = len(sp["rows"])
    for thr in (np.float32(wl.tau_mask), np.float32(wl.tau_edit)):
        assert np.abs(conf[:n] - float(thr)).min() >= 1e-3
    action, stats = O.t2t_update(sp["ocfg"], opk, sp["ost"], xhat, conf)
    ncom, spawned, ctr = O.gate_commit(sp["ocfg"], opk, stats, sp["ost"], sp["k_win"], sp["v_win"],
                                       sp["k_pool"], sp["v_pool"])
    rows = torch.from_numpy(sp["rows"]).to(DEV)
    np.testing.assert_array_equal(sb.argmax[rows].cpu().numpy(), xhat[:n])
    np.testing.assert_allclose(sb.conf[rows].cpu().numpy(), conf[:n], rtol=0, atol=2e-5)
    np.testing.assert_array_equal(sb.action[rows].cpu().numpy(), action[:n])
    assert (action[:n] == O.ACT_M2T).any() and (action[:n] == O.ACT_T2T).any()
    slots = (sp["rows"][::wl.block_len] // wl.block_len).astype(np.int64)
    np.testing.assert_array_equal(sb.slot_stats.cpu().numpy()[slots], stats[:len(slots)])
    g = longctx["st"].to_numpy()
    for r in longctx["keep"]:
        assert int(sb.n_committed[r]) == int(ncom[r]) and int(sb.spawned[r]) == int(spawned[r])
        for name in ("active", "prefix_len", "L", "R"):
            assert int(g[name][r]) == int(getattr(sp["ost"], name)[r]), (name, r)
        np.testing.assert_array_equal(g["pe_done"][r], sp["ost"].pe_done[r])
        np.testing.assert_array_equal(g["tokens"][r], sp["ost"].tokens[r])
    c = sb.step_counters.cpu().numpy()
    assert c[O.CT_BLOCKS] == int(sb.n_committed.sum()) and c[O.CT_SPAWNED] == int(sb.spawned.sum())
    assert c[O.CT_LIVE_SLOTS] == longctx["n_live"]


@pytest.mark.parametrize("shape", ["longctx_32768_w3", "batch64_65536_w4"])
def test_single_long_request_runs_entirely_as_split_pieces(shape):
    """One decoding request with a very long prefix and nothing else in the
    batch: every unit of the work list is cut along the key axis (the case that
    drives the number of partial results to its bound; eight query heads keep
    the oracle at seconds).  All rows against the oracle; the work list on the
    device against the host-side plan."""
    import dataclasses
    if shape == "longctx_32768_w3":
        wl = dataclasses.replace(synth.WORKLOADS[3], n_requests=4, prefix_lo=32768, prefix_hi=32768,
                                 n_q_heads=8, n_kv_heads=2)
    else:
        wl = dataclasses.replace(synth.WORKLOADS[2], n_requests=4, prefix_lo=65536, prefix_hi=65536,
                                 w_lo=4, w_hi=4, n_q_heads=8, n_kv_heads=2)
    stc = synth.make_structure(wl, n_inactive=wl.n_requests - 1)
    tokens = synth.make_tokens(stc)
    attn = synth.make_attn_inputs(stc)
    ctx = B.Context(**synth.config_dict(stc))
    st = B.DeviceState.from_numpy(DEV, stc.active, stc.prefix_len, stc.L, stc.R, tokens,
                                  np.zeros((wl.n_requests, wl.wmax), np.uint8), stc.page_table)
    pk = B.PackBuffers.alloc(ctx, DEV)
    sb = B.StepBuffers(ctx, DEV)
    q, kw, vw, kp, vp = (t.to(DEV) for t in attn)
    sb.out.fill_(7.0)
    B.fb_pack_wavefronts(ctx, st, pk, sb.ws, sb.status)
    B.fb_wavefront_attn(ctx, pk, q, kw, vw, kp, vp, st.page_table, sb.out, sb.ws, sb.status)
    torch.cuda.synchronize()
    assert int(sb.status.item()) == 0
    hdr = sb.ws[:64].cpu().numpy().view(np.int32)          # n_items, n_units, chunk length, n_parts
    act = stc.active == 1
    plan = ctx.attn_plan(stc.prefix_len[act], (stc.R - stc.L)[act])
    assert (int(hdr[1]), int(hdr[0]), int(hdr[3])) == (plan["units"], plan["items"], plan["parts"])
    assert plan["parts"] == plan["items"] > plan["units"], "every unit was meant to be split"
    assert plan["parts"] <= plan["max_parts"]
    ocfg = H.oracle_cfg(stc)
    opk = O.pack_wavefronts(ocfg, H.oracle_state(stc, tokens))
    ref = O.wavefront_attn(ocfg, opk, *(H.f64(t) for t in attn), stc.page_table)
    rows = H.live_rows(opk, wl.block_len)
    max_abs, rel = H.attn_errors(sb.out, ref, rows)
    assert max_abs <= 1e-2 and rel <= 5e-3, (max_abs, rel)
    assert bool((sb.out[len(rows):].float() == 7.0).all())


@pytest.mark.parametrize("window_in_pages", [0, 1])
def test_serving_structure_attention_sampled_requests(window_in_pages):
    """The serving workload's structure at full size (128 requests, 512 slots of
    capacity, prefixes of 512-4096 tokens, one to four live blocks each): the
    packing of all requests bit for bit, the attention of four sampled requests
    (first, last, and the ones with the shortest and the longest prefix)
    against the oracle; also with the window resident in the pages (Eq. 6
    scatter first, every key read through the page table)."""
    wl = synth.WORKLOADS[4]
    stc = synth.make_structure(wl)
    tokens = synth.make_tokens(stc)
    attn = synth.make_attn_inputs(stc)
    ctx = B.Context(**synth.config_dict(stc, window_in_pages=window_in_pages))
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
    assert int(sb.status.item()) == 0
    ocfg = O.Config(**synth.config_dict(stc))
    opk_all = O.pack_wavefronts(ocfg, H.oracle_state(stc, tokens))
    g = pk.to_numpy()
    assert int(g["n_live"][0]) == opk_all.n_live
    for name in ("slot_req", "slot_s", "slot_pos0", "slot_kv_len", "slot_flags", "req_slot_begin", "qtok", "pos"):
        np.testing.assert_array_equal(g[name], getattr(opk_all, name), err_msg=name)
    keep = sorted({0, wl.n_requests - 1, int(np.argmin(stc.prefix_len)), int(np.argmax(stc.prefix_len))})
    sp = H.sub_problem(stc, tokens, attn, None, keep)
    opk = O.pack_wavefronts(sp["ocfg"], sp["ost"])
    ref = O.wavefront_attn(sp["ocfg"], opk, sp["q"], sp["k_win"], sp["v_win"], sp["k_pool"], sp["v_pool"],
                           sp["ost"].page_table)
    n = len(sp["rows"])
    got = sb.out[torch.from_numpy(sp["rows"]).to(DEV)].float().cpu().numpy().astype(np.float64)
    err = np.abs(got - ref[:n])
    rel = np.linalg.norm(got - ref[:n]) / np.linalg.norm(ref[:n])
    assert err.max() <= 1e-2 and rel <= 5e-3, (err.max(), rel)
    live = synth.n_live_slots(stc) * wl.block_len
    assert bool(torch.isfinite(sb.out[:live].float()).all())
    assert bool((sb.out[live:].float() == 7.0).all())


def test_lm_head_fused_row_pass_full_vocabulary_sampled_rows():
    """The fused LM head at the benchmark's size (4,768 live rows, V = 151,552,
    hidden 2048): winners and confidences of sampled rows against the oracle's
    plain x W^T followed by its row pass; all rows against properties."""
    wl = synth.WORKLOADS[2]
    stc = synth.make_structure(wl)
    tokens = synth.make_tokens(stc)
    hidden = 2048
    rows = wl.max_slots * wl.block_len
    n_live = synth.n_live_slots(stc)
    live = n_live * wl.block_len
    w = synth.randn_bf16((wl.vocab, hidden), stc.seed, 13, 1.0 / np.sqrt(hidden))
    x = synth.randn_bf16((rows, hidden), stc.seed, 14)
    rg = np.random.default_rng(17)
    sample = np.sort(rg.choice(live, size=24, replace=False))
    sample[0], sample[-1] = 0, live - 1                     # first and last live row (ragged last row tile)
    winners = rg.integers(0, wl.vocab - 2, size=len(sample))
    for i, wi in zip(sample, winners):                      # a clear winner with a confidence around 0.5-0.95
        wv = w[wi].to(torch.float64)
        boost = rg.uniform(12.5, 15.5)
        x[i] = (x[i].to(torch.float64) + boost * wv / float(wv @ wv)).to(torch.bfloat16)
    ctx = B.Context(**synth.config_dict(stc))
    st = B.DeviceState.from_numpy(DEV, stc.active, stc.prefix_len, stc.L, stc.R, tokens,
                                  np.zeros((wl.n_requests, wl.wmax), np.uint8), stc.page_table)
    pk = B.PackBuffers.alloc(ctx, DEV)
    sb = B.StepBuffers(ctx, DEV)
    ws = torch.zeros(B.lib().fb_lm_head_workspace_bytes(ctx.handle), dtype=torch.uint8, device=DEV)
    B.fb_pack_wavefronts(ctx, st, pk, sb.ws, sb.status)
    B.fb_lm_head_t2t(ctx, pk, x.to(DEV), w.to(DEV), st, sb.argmax, sb.conf, sb.action, sb.slot_stats, ws,
                     sb.status)
    torch.cuda.synchronize()
    assert int(sb.status.item()) == 0
    # oracle on the sampled rows, packed as the live rows of a small problem of its own
    import dataclasses
    b = wl.block_len
    n_slots = (len(sample) + b - 1) // b
    mini = dataclasses.replace(wl, n_requests=n_slots, wmax=1, w_lo=1, w_hi=1, prefix_lo=0, prefix_hi=0,
                               max_blocks=2)
    mstc = synth.make_structure(mini)
    mcfg = H.oracle_cfg(mstc)
    mpk = O.pack_wavefronts(mcfg, H.oracle_state(mstc, synth.make_tokens(mstc)))
    assert mpk.n_live == n_slots
    xs = np.zeros((n_slots * b, hidden))
    xs[:len(sample)] = H.f64(x[torch.from_numpy(sample)])
    # x W^T in slices of the vocabulary (W in fp64 would not fit at once), then the oracle's row pass
    z_all = []
    for v0 in range(0, wl.vocab, 16384):
        z_all.append(xs @ H.f64(w[v0:v0 + 16384]).T)
    z = np.concatenate(z_all, axis=1)
    full_logits = np.zeros((mcfg.max_slots * b, wl.vocab))
    full_logits[:n_slots * b] = z
    xo, co = O.t2t_rows(mcfg, mpk, full_logits)
    got_a = sb.argmax.cpu().numpy()[sample]
    got_c = sb.conf.cpu().numpy()[sample].astype(np.float64)
    np.testing.assert_array_equal(got_a, xo[:len(sample)])
    np.testing.assert_array_equal(got_a, winners)
    assert np.abs(got_c - co[:len(sample)]).max() <= 2e-4, np.abs(got_c - co[:len(sample)]).max()
    assert co[:len(sample)].min() > 0.05 and co[:len(sample)].max() > 0.9
    # every live row: a token inside the vocabulary, a probability; padding rows as in fb_t2t_step
    am, cf = sb.argmax.cpu().numpy(), sb.conf.cpu().numpy()
    assert ((am[:live] >= 0) & (am[:live] < wl.vocab)).all() and ((cf[:live] > 0) & (cf[:live] <= 1)).all()
    assert (am[live:] == -1).all() and not cf[live:].any()


def test_fp8_pages_attention_sampled_requests_at_the_bench_size():
    """The 8-bit-page attention at the benchmark's size (64 requests, prefixes
    1K-8K): scatter (quantiser) + attention, six sampled requests against the
    oracle with the tolerance tests/test_gpu_fp8.py derives (rel-L2 at most 1.5 x
    3.75e-2; element-wise 6 standard deviations of the row's rounding error
    plus the bf16 output's 1e-2)."""
    wl = synth.WORKLOADS[2]
    stc = synth.make_structure(wl)
    tokens = synth.make_tokens(stc)
    q, kw, vw, _, _ = synth.make_attn_inputs(stc)
    k8, v8, ks, vs = synth.make_fp8_kv(stc)
    ctx = B.Context(kv_fp8=1, **synth.config_dict(stc, window_in_pages=1))
    st = B.DeviceState.from_numpy(DEV, stc.active, stc.prefix_len, stc.L, stc.R, tokens,
                                  np.zeros((wl.n_requests, wl.wmax), np.uint8), stc.page_table)
    pk = B.PackBuffers.alloc(ctx, DEV)
    sb = B.StepBuffers(ctx, DEV)
    dk8, dv8, dks, dvs = k8.to(DEV), v8.to(DEV), ks.to(DEV), vs.to(DEV)
    sb.out.fill_(7.0)
    B.fb_pack_wavefronts(ctx, st, pk, sb.ws, sb.status)
    B.fb_scatter_window_kv_fp8(ctx, pk, st.page_table, kw.to(DEV), vw.to(DEV), dk8, dv8, dks, dvs, sb.status)
    B.fb_wavefront_attn_fp8(ctx, pk, q.to(DEV), dk8, dv8, dks, dvs, st.page_table, sb.out, sb.ws, sb.status)
    torch.cuda.synchronize()
    assert int(sb.status.item()) == 0
    order = np.argsort(stc.prefix_len)
    keep = sorted({int(order[0]), int(order[-1]), int(np.argmax(stc.R - stc.L)), 5, 23, 41})
    # the sampled requests as a problem of their own; the 8-bit pools go through the same page remap
    # as bf16 tensors of code values (sub_problem only moves rows around), then back to bytes
    as_bf16 = lambda t8: t8.to(torch.float32).to(torch.bfloat16)        # codes 0..255 are exact in bf16
    sp = H.sub_problem(stc, tokens, (q, kw, vw, as_bf16(k8), as_bf16(v8)), None, keep)
    opk = O.pack_wavefronts(sp["ocfg"], sp["ost"])
    ok8, ov8 = sp["k_pool"].astype(np.uint8), sp["v_pool"].astype(np.uint8)
    O.scatter_window_kv_fp8(sp["ocfg"], opk, sp["k_win"], sp["v_win"], ok8, ov8, ks.numpy(), vs.numpy(),
                            sp["ost"].page_table)
    ref = O.wavefront_attn_fp8(sp["ocfg"], opk, sp["q"], ok8, ov8, ks.numpy(), vs.numpy(), sp["ost"].page_table)
    n = len(sp["rows"])
    got = sb.out[torch.from_numpy(sp["rows"]).to(DEV)].float().cpu().numpy().astype(np.float64)
    rel = np.linalg.norm(got - ref[:n]) / np.linalg.norm(ref[:n])
    kd = O.e4m3_decode(ok8) * ks.numpy()[None, :, None, None]
    n2 = O.wavefront_attn_weight_norms(sp["ocfg"], opk, sp["q"], None, kd, sp["ost"].page_table)
    allowed = 6.0 * 3.75e-2 * np.sqrt(n2[:n])[:, :, None] + 1e-2
    worst = float((np.abs(got - ref[:n]) / allowed).max())
    assert rel <= 1.5 * 3.75e-2 and worst <= 1.0, (rel, worst)
    live = synth.n_live_slots(stc) * wl.block_len
    assert bool(torch.isfinite(sb.out[:live].float()).all())
    assert bool((sb.out[live:].float() == 7.0).all())
