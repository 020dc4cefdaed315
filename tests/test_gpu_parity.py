"""GPU parity: every C-ABI call against the fp64 oracle on the same seeded
inputs, element by element.  Integer / index / decision outputs must be
bit-exact; confidence within 2e-5 absolute (fp32 sum of up to 151,552 terms
with ex2.approx in about 2,400 partial sums: relative error below 1e-6);
attention within max-abs 1e-2 and relative L2 5e-3 of the oracle (bf16 inputs,
fp32 accumulation, bf16 output)."""
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
CONF_TOL = 2e-5
ATTN_MAX_ABS, ATTN_REL_L2 = 1e-2, 5e-3
MARGIN = 1e-3


def make_case(wl, seed=None, n_inactive=0, logits_kind=None, conf_shift=0.0,
              with_attn=True, with_logits=True):
    stc = synth.make_structure(wl, seed, n_inactive=n_inactive)
    tokens = synth.make_tokens(stc)
    case = dict(wl=wl, stc=stc)
    if with_logits:
        z, tokens = synth.make_logits(stc, tokens, logits_kind,
                                      conf_shift=conf_shift)
        case["logits"] = z
    case["tokens"] = tokens
    if with_attn:
        case["attn"] = synth.make_attn_inputs(stc)
    return case


def gpu_objects(case, **over):
    stc = case["stc"]
    ctx = B.Context(**H.common_cfg(stc, **over))
    st = B.DeviceState.from_numpy(
        DEV, stc.active, stc.prefix_len, stc.L, stc.R, case["tokens"],
        np.zeros((stc.wl.n_requests, stc.wl.wmax), np.uint8), stc.page_table)
    pk = B.PackBuffers.alloc(ctx, DEV)
    sb = B.StepBuffers(ctx, DEV)
    return ctx, st, pk, sb


def check_pack(pk_gpu: B.PackBuffers, pk: O.Pack):
    g = pk_gpu.to_numpy()
    assert int(g["n_live"][0]) == pk.n_live
    for name in ("slot_req", "slot_s", "slot_pos0", "slot_kv_len",
                 "slot_flags", "req_slot_begin", "qtok", "pos"):
        np.testing.assert_array_equal(g[name], getattr(pk, name), err_msg=name)


WORKLOADS = {
    "tiny": synth.tiny_workload(),
    "tiny_d128_b64": synth.tiny_workload(head_dim=128, block_len=64, wmax=3,
                                         n_q_heads=8, n_kv_heads=2,
                                         prefix_lo=0, prefix_hi=700),
    "tiny_wide": synth.tiny_workload(n_requests=9, wmax=4, n_q_heads=4,
                                     n_kv_heads=1, prefix_lo=120,
                                     prefix_hi=136, w_lo=1, w_hi=4),
    "tiny_noprefix": synth.tiny_workload(prefix_lo=0, prefix_hi=0, w_lo=1,
                                         w_hi=3, n_requests=4),
    # block lengths 96 / 128 and W = 5 of the paper's robustness sweeps
    # (Sec. 4.5, 4.6), group sizes 8 and 1
    "tiny_b96": synth.tiny_workload(block_len=96, wmax=2, w_lo=1, w_hi=2,
                                    n_q_heads=8, n_kv_heads=2, head_dim=128,
                                    prefix_lo=0, prefix_hi=500, n_requests=4),
    "tiny_b128_w5_mha": synth.tiny_workload(block_len=128, wmax=5, w_lo=1, w_hi=5,
                                            n_q_heads=2, n_kv_heads=2, head_dim=64,
                                            prefix_lo=3, prefix_hi=260, n_requests=4,
                                            max_blocks=16),
    "tiny_g8": synth.tiny_workload(n_q_heads=16, n_kv_heads=2, head_dim=128,
                                   prefix_lo=60, prefix_hi=420, n_requests=4),
    # a vocabulary whose 16-byte pieces (125) do not divide among the two CTAs of a row
    "tiny_v1000": synth.tiny_workload(vocab=1000),
    "cfg0": synth.WORKLOADS[0],
    "cfg1": synth.WORKLOADS[1],
}


# ------------------------------------------------------------------- pack
@pytest.mark.parametrize("name", list(WORKLOADS))
@pytest.mark.parametrize("n_inactive", [0, 1])
def test_pack_bit_exact(name, n_inactive):
    wl = WORKLOADS[name]
    if n_inactive >= wl.n_requests:
        pytest.skip("single request")
    case = make_case(wl, n_inactive=n_inactive, with_attn=False,
                     with_logits=False)
    ctx, st, pk, sb = gpu_objects(case)
    B.fb_pack_wavefronts(ctx, st, pk, sb.ws, sb.status)
    torch.cuda.synchronize()
    ref = O.pack_wavefronts(H.oracle_cfg(case["stc"]),
                            H.oracle_state(case["stc"], case["tokens"]))
    check_pack(pk, ref)
    assert int(sb.status.item()) == 0


def test_pack_empty_and_full_batches():
    wl = synth.tiny_workload(n_requests=5, wmax=4, w_lo=4, w_hi=4)
    case = make_case(wl, with_attn=False, with_logits=False)
    stc = case["stc"]
    for active in (np.zeros(5, np.int32), np.ones(5, np.int32),
                   np.array([2, 1, 0, 1, 2], np.int32)):
        stc.active[:] = active
        ctx, st, pk, sb = gpu_objects(case)
        B.fb_pack_wavefronts(ctx, st, pk, sb.ws, sb.status)
        torch.cuda.synchronize()
        ref = O.pack_wavefronts(H.oracle_cfg(stc), H.oracle_state(stc, case["tokens"]))
        check_pack(pk, ref)
        assert ref.n_live == 4 * int((active == 1).sum())


def test_pack_flags_corrupt_state_without_faulting():
    wl = synth.tiny_workload(n_requests=4, wmax=2, w_lo=1, w_hi=2)
    case = make_case(wl, with_attn=False, with_logits=False)
    case["stc"].R[1] = case["stc"].L[1] + 5            # window wider than W
    ctx, st, pk, sb = gpu_objects(case)
    B.fb_pack_wavefronts(ctx, st, pk, sb.ws, sb.status)
    torch.cuda.synchronize()
    assert int(sb.status.item()) & B.FB_ST_BAD_STATE
    assert int(pk.n_live.item()) <= ctx.max_slots


# -------------------------------------------------------------------- T2T
def run_t2t_and_gate(case, **over):
    stc = case["stc"]
    ctx, st, pk, sb = gpu_objects(case, **over)
    z = case["logits"].to(DEV)
    attn = case.get("attn")
    if attn is not None:
        q, kw, vw, kp, vp = (t.to(DEV) for t in attn)
    else:
        wl = stc.wl
        kw = torch.zeros(ctx.max_slots * wl.block_len, wl.n_kv_heads, wl.head_dim,
                         dtype=torch.bfloat16, device=DEV)
        vw = torch.zeros_like(kw)
        kp = torch.zeros(stc.num_pages, wl.n_kv_heads, 64, wl.head_dim,
                         dtype=torch.bfloat16, device=DEV)
        vp = torch.zeros_like(kp)
    B.fb_pack_wavefronts(ctx, st, pk, sb.ws, sb.status)
    B.fb_t2t_step(ctx, pk, z, st, sb.argmax, sb.conf, sb.action, sb.slot_stats,
                  sb.status)
    torch.cuda.synchronize()
    tokens_after_t2t = st.tokens.cpu().numpy().copy()
    B.fb_gate_commit(ctx, pk, sb.slot_stats, st, kw, vw, kp, vp, sb.n_committed,
                     sb.spawned, sb.step_counters, sb.status)
    torch.cuda.synchronize()
    # oracle
    ocfg = H.oracle_cfg(stc, **over)
    ost = H.oracle_state(stc, case["tokens"])
    opk = O.pack_wavefronts(ocfg, ost)
    xhat, conf = O.t2t_rows(ocfg, opk, H.f64(case["logits"]))
    live = opk.n_live * stc.wl.block_len
    for thr in (np.float32(ocfg.tau_mask), np.float32(ocfg.tau_edit)):
        assert np.abs(conf[:live] - float(thr)).min() >= MARGIN, \
            "generator left a confidence inside the decision margin"
    tokens_before = ost.tokens.copy()
    action, stats = O.t2t_update(ocfg, opk, ost, xhat, conf)
    forced_margin = forced_reveal_margin(ocfg, opk, ost, tokens_before, action, conf)
    np.testing.assert_array_equal(sb.argmax.cpu().numpy(), xhat)
    np.testing.assert_allclose(sb.conf.cpu().numpy(), conf, rtol=0, atol=CONF_TOL)
    np.testing.assert_array_equal(sb.action.cpu().numpy(), action)
    np.testing.assert_array_equal(sb.slot_stats.cpu().numpy(), stats)
    np.testing.assert_array_equal(tokens_after_t2t, ost.tokens)
    if attn is not None:
        okw, ovw, okp, ovp = (H.f64(t) for t in attn[1:])
        kvargs = (okw, ovw, okp, ovp)
    else:
        kvargs = ()
    ncom, spawned, ctr = O.gate_commit(ocfg, opk, stats, ost, *kvargs)
    np.testing.assert_array_equal(sb.n_committed.cpu().numpy(), ncom)
    np.testing.assert_array_equal(sb.spawned.cpu().numpy(), spawned)
    np.testing.assert_array_equal(sb.step_counters.cpu().numpy(), ctr)
    g = st.to_numpy()
    for name in ("active", "prefix_len", "L", "R", "tokens", "pe_done"):
        np.testing.assert_array_equal(g[name], getattr(ost, name), err_msg=name)
    if attn is not None:
        # pool pages: committed rows equal the window rows byte for byte,
        # everything else untouched
        np.testing.assert_array_equal(H.f64(kp.cpu()), okp)
        np.testing.assert_array_equal(H.f64(vp.cpu()), ovp)
    assert int(sb.status.item()) == 0
    return dict(action=action, stats=stats, ncom=ncom, spawned=spawned, ctr=ctr, forced_margin=forced_margin)


def forced_reveal_margin(ocfg, opk, ost, tokens_before, action, conf):
    """Smallest gap between the confidence of a force-revealed position and the
    best other masked position of its block (inf if nothing was forced)."""
    b = ocfg.block_len
    gap = np.inf
    for i in np.flatnonzero(action == O.ACT_FORCED):
        slot, r = i // b, int(opk.slot_req[i // b])
        L_before = int(ost.L[r])          # t2t_update does not move L
        g = L_before + int(opk.slot_s[slot])
        masked = tokens_before[r, g * b:(g + 1) * b] == ocfg.mask_id
        others = [conf[slot * b + t] for t in range(b) if masked[t] and slot * b + t != i]
        if others:
            gap = min(gap, float(conf[i] - max(others)))
    return gap


@pytest.mark.parametrize("name,kind,shift,s_pe", [
    ("tiny", "calibrated", 0.0, 1), ("tiny", "calibrated", 0.3, 0),
    ("tiny_wide", "calibrated", 0.2, 1), ("tiny_d128_b64", "calibrated", 0.1, 3),
    ("tiny", "literal", 0.0, 1), ("cfg0", "normal2", 0.0, 1), ("tiny_v1000", "calibrated", 0.1, 1)])
def test_t2t_and_gate_commit_bit_exact(name, kind, shift, s_pe):
    # the shifted case runs on a seed whose draw retires a block within this one step (most draws
    # leave at least one mask in every oldest block)
    case = make_case(WORKLOADS[name], seed=101 if shift >= 0.3 else None, logits_kind=kind, conf_shift=shift)
    res = run_t2t_and_gate(case, s_pe=s_pe)
    if kind == "calibrated":
        assert (res["action"] == O.ACT_M2T).any() and (res["action"] == O.ACT_T2T).any()
    if shift >= 0.3:
        assert res["ncom"].sum() >= 1, "the shifted confidences were meant to commit at least one block"


@pytest.mark.parametrize("name,shift,s_pe", [("tiny", 0.3, 0), ("tiny_wide", 0.2, 1),
                                             ("tiny_d128_b64", 0.1, 3)])
def test_t2t_and_batch_synchronous_gate_bit_exact(name, shift, s_pe):
    """The whole step with fb_config.batch_sync = 1 (Sec. 3.2: all()-gated
    retirement, min-rho admission)."""
    case = make_case(WORKLOADS[name], logits_kind="calibrated", conf_shift=shift)
    run_t2t_and_gate(case, s_pe=s_pe, batch_sync=1)


@pytest.mark.parametrize("batch_sync", [0, 1])
@pytest.mark.parametrize("seed", range(12))
def test_gate_commit_on_drawn_block_counts(seed, batch_sync):
    """fb_gate_commit alone on block counts drawn from a menu (finished,
    finished with EOS, half ready, a quarter ready, fully masked) over drawn
    windows, so that cascades, committed EOS, sequences running out of blocks,
    stragglers and every admission outcome occur; per-sequence and
    batch-synchronous policy, bit-exact against the oracle, K/V freeze included."""
    rg = np.random.default_rng(500 + seed)
    _gate_commit_case(rg, seed, batch_sync, int(rg.integers(1, 10)), int(rg.integers(1, 5)))


@pytest.mark.parametrize("batch_sync", [0, 1])
@pytest.mark.parametrize("Rn,W,seed", [(128, 4, 3), (600, 2, 4), (600, 3, 8)])
def test_gate_commit_on_drawn_block_counts_many_requests(Rn, W, seed, batch_sync):
    """The same with more requests than the reduction kernel has threads
    (seeds 4 and 8 start from a shared window)."""
    _gate_commit_case(np.random.default_rng(700 + seed), seed, batch_sync, Rn, W)


def _gate_commit_case(rg, seed, batch_sync, Rn, W):
    n = 6
    wl = synth.tiny_workload(n_requests=Rn, wmax=W, w_lo=1, w_hi=W, max_blocks=n,
                             n_q_heads=8, n_kv_heads=2, prefix_lo=0, prefix_hi=90)
    case = make_case(wl, seed=900 + seed, with_logits=False)
    stc = case["stc"]
    b = wl.block_len
    # windows anywhere in [0, n], some empty, some touching n, some requests idle or done
    for r in range(Rn):
        L = int(rg.integers(0, n + 1))
        stc.L[r] = L
        stc.R[r] = min(n, L + int(rg.integers(0, W + 1)))
        stc.active[r] = rg.choice([0, 1, 1, 1, 1, 2])
    if seed % 4 == 0:                      # a shared window: the ablation's own setting
        stc.L[:] = 2; stc.R[:] = min(n, 2 + W); stc.active[:] = 1
    over = dict(batch_sync=batch_sync, s_pe=int(rg.integers(0, 3)),
                theta_spawn=float(rg.choice([0.25, 0.5, 0.6])))
    ctx, st, pk, sb = gpu_objects(case, **over)
    pe0 = rg.integers(0, 3, size=(Rn, W)).astype(np.uint8)
    st.pe_done.copy_(torch.from_numpy(pe0))
    q, kw, vw, kp, vp = (t.to(DEV) for t in case["attn"])
    B.fb_pack_wavefronts(ctx, st, pk, sb.ws, sb.status)
    torch.cuda.synchronize()
    ocfg = H.oracle_cfg(stc, **over)
    ost = H.oracle_state(stc, case["tokens"])
    ost.pe_done[:] = pe0
    opk = O.pack_wavefronts(ocfg, ost)
    menu = np.array([(0, 0, 0, 0, 0, 0), (0, 0, 0, 0, 0, 1), (b, b // 2, 0, 0, b, 0),
                     (b, b // 4, 0, 0, b, 0), (b, 0, 0, 0, b, 0), (3, 3, 3, 0, 0, 0),
                     (0, 0, 0, 2, 0, 0)], np.int32)
    weights = [0.45, 0.08, 0.12, 0.1, 0.1, 0.1, 0.05]
    stats = np.zeros((ctx.max_slots, 6), np.int32)
    stats[:opk.n_live] = menu[rg.choice(len(menu), size=opk.n_live, p=weights)]
    sb.slot_stats.copy_(torch.from_numpy(stats))
    B.fb_gate_commit(ctx, pk, sb.slot_stats, st, kw, vw, kp, vp, sb.n_committed, sb.spawned,
                     sb.step_counters, sb.status)
    torch.cuda.synchronize()
    okw, ovw, okp, ovp = (H.f64(t) for t in case["attn"][1:])
    ncom, spawned, ctr = O.gate_commit(ocfg, opk, stats, ost, okw, ovw, okp, ovp)
    np.testing.assert_array_equal(sb.n_committed.cpu().numpy(), ncom)
    np.testing.assert_array_equal(sb.spawned.cpu().numpy(), spawned)
    np.testing.assert_array_equal(sb.step_counters.cpu().numpy(), ctr)
    g = st.to_numpy()
    for name in ("active", "prefix_len", "L", "R", "tokens", "pe_done"):
        np.testing.assert_array_equal(g[name], getattr(ost, name), err_msg=name)
    np.testing.assert_array_equal(H.f64(kp.cpu()), okp)
    np.testing.assert_array_equal(H.f64(vp.cpu()), ovp)
    assert int(sb.status.item()) == 0


@pytest.mark.parametrize("name,shift,thr,over", [
    ("tiny", 0.0, (0.9, 0.6), dict(delta_literal=1)),
    ("tiny_wide", 0.2, (0.95, 0.9), dict(delta_literal=1)),
    ("tiny", 0.3, (0.9, 0.95), dict(delta_literal=1)),                       # usual order: no effect
    ("tiny", -0.4, (0.9, 0.95), dict(force_progress=1)),
    ("tiny_wide", -0.3, (0.9, 0.95), dict(force_progress=1, s_pe=0)),
    ("tiny_d128_b64", -0.5, (0.9, 0.85), dict(force_progress=1, delta_literal=1)),
    ("tiny_wide", -0.3, (0.9, 0.95), dict(force_progress=1, batch_sync=1))])
def test_update_modes_bit_exact(name, shift, thr, over):
    """Eq. 1 with Delta taken literally and / or the forced-progress rule on the
    oldest block, whole T2T + gate step against the oracle.  The thresholds go
    into the workload so that the generator keeps its margin around them."""
    wl = dataclasses.replace(WORKLOADS[name], tau_mask=thr[0], tau_edit=thr[1])
    for seed in range(20):
        case = make_case(wl, seed=synth.BASE_SEED + 700 + seed, logits_kind="calibrated", conf_shift=shift)
        if not over.get("force_progress"):
            break
        # a forced reveal compares confidences with each other: take a draw (judged by the
        # oracle alone) in which no such comparison is closer than the decision margin
        stc = case["stc"]
        ocfg = H.oracle_cfg(stc, **over)
        ost = H.oracle_state(stc, case["tokens"])
        opk = O.pack_wavefronts(ocfg, ost)
        xhat, conf = O.t2t_rows(ocfg, opk, H.f64(case["logits"]))
        before = ost.tokens.copy()
        action, _ = O.t2t_update(ocfg, opk, ost, xhat, conf)
        if (action == O.ACT_FORCED).any() and forced_reveal_margin(ocfg, opk, ost, before, action, conf) >= MARGIN:
            break
    else:
        pytest.fail("no draw with a forced reveal outside the decision margin")
    res = run_t2t_and_gate(case, **over)
    if over.get("force_progress"):
        assert (res["action"] == B.FB_ACT_FORCED).any(), "no block needed the forced reveal in this draw"
        # the reveal is decided by comparing confidences: the draw must not hinge on the last bits
        assert res["forced_margin"] >= MARGIN
    if thr[1] < thr[0] and shift >= 0:
        assert (res["action"] == O.ACT_M2T).any()


def test_t2t_full_vocab_rows():
    """V = 151,552 rows: many tiles per row, bf16 ties, peaked rows."""
    wl = dataclasses.replace(synth.WORKLOADS[1], n_requests=2, name="cfg1_2req")
    case = make_case(wl, logits_kind="calibrated", with_attn=False)
    res = run_t2t_and_gate(case)
    assert (res["action"] == O.ACT_M2T).any()


def test_t2t_hand_worked_rows():
    """Closed-form rows 'one logit = a, others 0' (p = e^a / (e^a + V - 1)),
    exact ties, and the Eq. 1 / Eq. 2 / Eq. 3 hand-worked block."""
    V, b = 8, 32
    wl = synth.tiny_workload(n_requests=1, wmax=2, w_lo=1, w_hi=1, vocab=V,
                             n_q_heads=4, n_kv_heads=1, max_blocks=4)
    stc = synth.make_structure(wl)
    stc.L[:] = 0; stc.R[:] = 1
    stc.mask_id, stc.eos_id = 9, 10
    tokens = np.full((1, wl.max_blocks * b), 9, np.int32)
    tokens[0, :b] = ([9, 9, 3, 0] * 8)
    z = torch.zeros(wl.max_slots * b, V)
    spec = [(2, 5.0), (1, 3.0), (1, 5.0), (3, 4.0)] * 8
    for i, (w, a) in enumerate(spec):
        z[i, w] = a
    z[5] = 0.0                                   # 8-way tie -> index 0, p = 1/8
    case = dict(wl=wl, stc=stc, tokens=tokens, logits=z.to(torch.bfloat16))
    res = run_t2t_and_gate(case, theta_spawn=0.5)
    a = res["action"][:b]
    assert list(a[:4]) == [O.ACT_M2T, O.ACT_NONE, O.ACT_T2T, O.ACT_NONE]
    assert res["spawned"][0] == 1 and res["ncom"][0] == 0


def test_step_replayed_from_a_cuda_graph_matches_direct_launches():
    """The step is shape-stable (grids depend on the slot capacity, the live
    count is read on the device), so one captured step can be replayed while
    the state moves under it: four replays against four directly launched
    steps, everything bit for bit (attention output included: the dynamic
    hand-out of work items does not change any item's arithmetic)."""
    wl = synth.tiny_workload(n_requests=5, wmax=3, w_lo=1, w_hi=2, max_blocks=12, prefix_lo=40, prefix_hi=700)
    case = make_case(wl, with_logits=False)
    # every row peaked (p ~ 0.9996): blocks reveal, get edited, retire and spawn at every step
    rows = wl.max_slots * wl.block_len
    zc = torch.zeros(rows, wl.vocab)
    win = torch.from_numpy(np.random.default_rng(3).integers(0, wl.vocab - 2, size=rows))
    zc[torch.arange(rows), win] = 14.0
    z = zc.to(torch.bfloat16).to(DEV)
    outs = []
    for use_graph in (False, True):
        ctx, st, pk, sb = gpu_objects(case, s_pe=0)
        q, kw, vw, kp, vp = (t.to(DEV) for t in case["attn"])

        def step():
            B.fb_pack_wavefronts(ctx, st, pk, sb.ws, sb.status)
            B.fb_wavefront_attn(ctx, pk, q, kw, vw, kp, vp, st.page_table, sb.out, sb.ws, sb.status)
            B.fb_t2t_step(ctx, pk, z, st, sb.argmax, sb.conf, sb.action, sb.slot_stats, sb.status)
            B.fb_gate_commit(ctx, pk, sb.slot_stats, st, kw, vw, kp, vp, sb.n_committed, sb.spawned,
                             sb.step_counters, sb.status)
        trace = []
        if use_graph:
            g = torch.cuda.CUDAGraph()
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                snap = {k: getattr(st, k).clone() for k in ("active", "prefix_len", "L", "R", "tokens", "pe_done")}
                pools = (kp.clone(), vp.clone())
                step()                                  # first call: device set-up happens outside the capture
                side.synchronize()
                for k, v in snap.items():
                    getattr(st, k).copy_(v)
                kp.copy_(pools[0]); vp.copy_(pools[1])
                side.synchronize()
                with torch.cuda.graph(g, stream=side):
                    step()
            torch.cuda.current_stream().wait_stream(side)
        for _ in range(4):
            g.replay() if use_graph else step()
            torch.cuda.synchronize()
            trace.append((sb.out.clone(), sb.action.clone(), sb.n_committed.clone(), sb.spawned.clone(),
                          sb.step_counters.clone(), st.tokens.clone(), st.L.clone(), st.R.clone(),
                          pk.n_live.clone()))
        assert int(sb.status.item()) == 0
        outs.append((trace, kp.clone(), vp.clone()))
    (ta, kpa, vpa), (tb, kpb, vpb) = outs
    for a, b in zip(ta, tb):
        live = int(a[8].item()) * wl.block_len
        assert torch.equal(a[0][:live], b[0][:live])
        for x, y in zip(a[1:], b[1:]):
            assert torch.equal(x, y)
    assert torch.equal(kpa, kpb) and torch.equal(vpa, vpb)
    assert sum(int(t[2].sum()) for t in ta) > 0, "nothing retired in four steps"


# -------------------------------------------------------------- attention
def run_attention(case, fill_pad=False, tuning=None):
    stc = case["stc"]
    wl = stc.wl
    ctx, st, pk, sb = gpu_objects(case, tuning=tuning)
    q, kw, vw, kp, vp = (t.to(DEV) for t in case["attn"])
    sb.out.fill_(7.0)
    B.fb_pack_wavefronts(ctx, st, pk, sb.ws, sb.status)
    B.fb_wavefront_attn(ctx, pk, q, kw, vw, kp, vp, st.page_table, sb.out,
                        sb.ws, sb.status)
    torch.cuda.synchronize()
    assert int(sb.status.item()) == 0, f"status {int(sb.status.item())}"
    ocfg = H.oracle_cfg(stc)
    opk = O.pack_wavefronts(ocfg, H.oracle_state(stc, case["tokens"]))
    ref = O.wavefront_attn(ocfg, opk, *(H.f64(t) for t in case["attn"]),
                           stc.page_table)
    rows = H.live_rows(opk, wl.block_len)
    max_abs, rel = H.attn_errors(sb.out, ref, rows)
    assert max_abs <= ATTN_MAX_ABS and rel <= ATTN_REL_L2, (max_abs, rel)
    # rows of padding slots are not written
    pad = sb.out[opk.n_live * wl.block_len:].float()
    assert bool((pad == 7.0).all())
    return max_abs, rel


@pytest.mark.parametrize("name", list(WORKLOADS))
def test_attention_matches_oracle(name):
    case = make_case(WORKLOADS[name], with_logits=False)
    run_attention(case)


@pytest.mark.parametrize("target", [1, 7, 100000])
def test_attention_split_kv_invariance(target):
    """Forcing very coarse / very fine key-axis splits changes nothing beyond
    rounding: the split is an execution detail."""
    wl = synth.tiny_workload(prefix_lo=900, prefix_hi=2600, n_requests=3,
                             head_dim=128, n_q_heads=8, n_kv_heads=2)
    case = make_case(wl, with_logits=False)
    run_attention(case, tuning=dict(attn_target_items=target))


def test_attention_isolation_from_invisible_memory():
    """Keys a query must not see (other requests, padding slots, pool rows
    beyond the prefix, blocks to the right) may hold anything finite."""
    wl = WORKLOADS["tiny"]
    case = make_case(wl, with_logits=False)
    stc = case["stc"]
    ocfg = H.oracle_cfg(stc)
    opk = O.pack_wavefronts(ocfg, H.oracle_state(stc, case["tokens"]))
    base = run_attention(case)
    q, kw, vw, kp, vp = (t.clone() for t in case["attn"])
    b = wl.block_len
    kw[opk.n_live * b:] = 300.0
    vw[opk.n_live * b:] = -300.0
    used = set()
    for r in range(wl.n_requests):
        if stc.active[r] != 1:
            continue
        P = int(stc.prefix_len[r])
        for j in range((P + 63) // 64):
            used.add(int(stc.page_table[r, j]))
        if P % 64:
            pg = int(stc.page_table[r, P // 64])
            kp[pg, :, P % 64:] = 250.0
            vp[pg, :, P % 64:] = -250.0
    for pg in range(stc.num_pages):
        if pg not in used:
            kp[pg] = 200.0
            vp[pg] = -200.0
    case2 = dict(case, attn=(q, kw, vw, kp, vp))
    again = run_attention(case2)
    assert again == base


def _amplify_keys(case, where, factor):
    """Returns attention inputs in which the keys of one stretch of every
    request's context are `factor` times larger, so that the running softmax
    reference has to move there: by a few powers of two (factor 6) or by far
    more than fp32's exponent range could absorb without re-basing (factor 40).
    V is halved so that near-one-hot outputs round to bf16 within the tolerance."""
    stc = case["stc"]
    wl = stc.wl
    b = wl.block_len
    q, kw, vw, kp, vp = (t.clone() for t in case["attn"])
    vw = (vw.float() * 0.5).to(torch.bfloat16)
    vp = (vp.float() * 0.5).to(torch.bfloat16)
    pk = O.pack_wavefronts(H.oracle_cfg(stc), H.oracle_state(stc, case["tokens"]))
    for r in range(wl.n_requests):
        if stc.active[r] != 1:
            continue
        P = int(stc.prefix_len[r])
        if where == "first_tile":
            lo, hi = 0, min(P, 100)
        elif where == "second_tile":
            lo, hi = min(P, 130), min(P, 250)
        elif where == "prefix_tail":
            lo, hi = max(P - 37, 0), P
        else:
            lo = hi = 0
        for pos in range(lo, hi):
            pg = int(stc.page_table[r, pos // 64])
            kp[pg, :, pos % 64] = (kp[pg, :, pos % 64].float() * factor).to(torch.bfloat16)
        if where == "window_last_block":
            s_last = int(pk.req_slot_begin[r + 1]) - 1
            rows = slice(s_last * b, (s_last + 1) * b)
            kw[rows] = (kw[rows].float() * factor).to(torch.bfloat16)
        if where == "window_first_block":
            s0 = int(pk.req_slot_begin[r])
            rows = slice(s0 * b, (s0 + 1) * b)
            kw[rows] = (kw[rows].float() * factor).to(torch.bfloat16)
    return q, kw, vw, kp, vp


@pytest.mark.parametrize("factor", [6.0, 40.0])
@pytest.mark.parametrize("where", ["first_tile", "second_tile", "prefix_tail",
                                   "window_first_block", "window_last_block"])
@pytest.mark.parametrize("target", [296, 100000])
def test_attention_when_the_softmax_reference_moves(where, factor, target):
    """Scores that jump far above (or start far above and fall far below) what
    earlier key tiles held: the lazily re-based reference, the rescaling of the
    accumulated output and the redo of the tile must agree with the plain
    softmax of the oracle, with and without a key-axis split."""
    wl = synth.tiny_workload(prefix_lo=300, prefix_hi=900, n_requests=5, wmax=4,
                             w_lo=1, w_hi=4, head_dim=128, n_q_heads=8, n_kv_heads=2,
                             max_blocks=16)
    case = make_case(wl, with_logits=False)
    case = dict(case, attn=_amplify_keys(case, where, factor))
    run_attention(case, tuning=dict(attn_target_items=target))


# --------------------------------------------------- multi-step state machine
def test_multi_step_trajectory_matches_oracle():
    """Eight consecutive steps (pack -> attention -> T2T -> gate/commit) with
    confidences rising by 0.05 per step and two requests arriving at steps 2
    and 4 (the serving-sweep pattern): states, pools and attention outputs are
    compared after every step, so commits and admissions of one step feed the
    next one on both sides."""
    wl = synth.tiny_workload(n_requests=5, wmax=3, w_lo=1, w_hi=2,
                             prefix_lo=40, prefix_hi=400, max_blocks=10)
    stc = synth.make_structure(wl, n_inactive=2)        # two requests arrive later
    late = [int(r) for r in np.flatnonzero(stc.active == 0)]
    tokens = synth.make_tokens(stc)
    case = dict(wl=wl, stc=stc, tokens=tokens)
    ctx, st, pk, sb = gpu_objects(case, s_pe=1)
    ocfg = H.oracle_cfg(stc, s_pe=1)
    ost = H.oracle_state(stc, tokens)
    q, kw, vw, kp, vp = synth.make_attn_inputs(stc)
    okp, ovp = H.f64(kp), H.f64(vp)
    dkp, dvp = kp.to(DEV), vp.to(DEV)
    total_commits = 0
    for step in range(8):
        if step in (2, 4):                  # staggered arrival: the caller writes the state row
            r = late[step // 2 - 1]
            ost.active[r] = 1
            st.active[r] = 1
        # this step's synthetic model outputs, placed from the ORACLE's state
        cur = dataclasses.replace(stc)
        cur.active, cur.prefix_len, cur.L, cur.R = (ost.active.copy(), ost.prefix_len.copy(),
                                                   ost.L.copy(), ost.R.copy())
        z, tok2 = synth.make_logits(cur, ost.tokens, "calibrated", seed_shift=step,
                                    conf_shift=0.05 * step)
        ost.tokens[:] = tok2
        st.tokens.copy_(torch.from_numpy(tok2))
        q = synth.randn_bf16(q.shape, stc.seed + step, 1)
        kw = synth.randn_bf16(kw.shape, stc.seed + step, 2)
        vw = synth.randn_bf16(vw.shape, stc.seed + step, 3)
        dq, dkw, dvw, dz = q.to(DEV), kw.to(DEV), vw.to(DEV), z.to(DEV)
        B.fb_pack_wavefronts(ctx, st, pk, sb.ws, sb.status)
        B.fb_wavefront_attn(ctx, pk, dq, dkw, dvw, dkp, dvp, st.page_table, sb.out, sb.ws, sb.status)
        B.fb_t2t_step(ctx, pk, dz, st, sb.argmax, sb.conf, sb.action, sb.slot_stats, sb.status)
        B.fb_gate_commit(ctx, pk, sb.slot_stats, st, dkw, dvw, dkp, dvp, sb.n_committed,
                         sb.spawned, sb.step_counters, sb.status)
        torch.cuda.synchronize()
        opk = O.pack_wavefronts(ocfg, ost)
        check_pack(pk, opk)
        ref = O.wavefront_attn(ocfg, opk, H.f64(q), H.f64(kw), H.f64(vw), okp, ovp, ost.page_table)
        max_abs, rel = H.attn_errors(sb.out, ref, H.live_rows(opk, wl.block_len))
        assert max_abs <= ATTN_MAX_ABS and rel <= ATTN_REL_L2, (step, max_abs, rel)
        xhat, conf = O.t2t_rows(ocfg, opk, H.f64(z))
        action, stats = O.t2t_update(ocfg, opk, ost, xhat, conf)
        ncom, spawned, ctr = O.gate_commit(ocfg, opk, stats, ost, H.f64(kw), H.f64(vw), okp, ovp)
        np.testing.assert_array_equal(sb.action.cpu().numpy(), action)
        np.testing.assert_array_equal(sb.n_committed.cpu().numpy(), ncom)
        np.testing.assert_array_equal(sb.spawned.cpu().numpy(), spawned)
        np.testing.assert_array_equal(sb.step_counters.cpu().numpy(), ctr)
        g = st.to_numpy()
        for name in ("active", "prefix_len", "L", "R", "tokens", "pe_done"):
            np.testing.assert_array_equal(g[name], getattr(ost, name), err_msg=f"{name}@{step}")
        np.testing.assert_array_equal(H.f64(dkp.cpu()), okp)
        np.testing.assert_array_equal(H.f64(dvp.cpu()), ovp)
        assert int(sb.status.item()) == 0
        total_commits += int(ncom.sum())
    assert total_commits >= 3, "the trajectory never committed a block"


def test_step_host_equals_the_four_calls():
    """fb_step_host (host buffers in, decisions out) against the four device
    calls on a second, identical state."""
    wl = synth.tiny_workload(n_requests=4, prefix_lo=30, prefix_hi=260)
    case = make_case(wl, logits_kind="calibrated", conf_shift=0.25)
    stc = case["stc"]
    q, kw, vw, kp, vp = case["attn"]
    z = case["logits"]
    # device path
    ctx, st, pk, sb = gpu_objects(case)
    dq, dkw, dvw, dkp, dvp, dz = (t.to(DEV) for t in (q, kw, vw, kp, vp, z))
    B.fb_pack_wavefronts(ctx, st, pk, sb.ws, sb.status)
    B.fb_wavefront_attn(ctx, pk, dq, dkw, dvw, dkp, dvp, st.page_table, sb.out, sb.ws, sb.status)
    B.fb_t2t_step(ctx, pk, dz, st, sb.argmax, sb.conf, sb.action, sb.slot_stats, sb.status)
    B.fb_gate_commit(ctx, pk, sb.slot_stats, st, dkw, dvw, dkp, dvp, sb.n_committed, sb.spawned,
                     sb.step_counters, sb.status)
    torch.cuda.synchronize()
    # host path on fresh buffers
    ctx2, st2, pk2, sb2 = gpu_objects(case)
    n_rows = synth.n_live_slots(stc) * wl.block_len
    hkp, hvp = kp.to(DEV), vp.to(DEV)
    dev = dict(q=torch.zeros_like(dq), k_win=torch.zeros_like(dkw), v_win=torch.zeros_like(dvw), out=sb2.out,
               logits=torch.zeros_like(dz), k_pool=hkp, v_pool=hvp, argmax=sb2.argmax, conf=sb2.conf,
               action=sb2.action, slot_stats=sb2.slot_stats, n_committed=sb2.n_committed, spawned=sb2.spawned,
               step_counters=sb2.step_counters, status=sb2.status, ws=sb2.ws)
    host = dict(h_q=q.pin_memory(), h_k_win=kw.pin_memory(), h_v_win=vw.pin_memory(), h_logits=z.pin_memory(),
                h_n_committed=torch.full((wl.n_requests,), -1, dtype=torch.int32).pin_memory(),
                h_spawned=torch.full((wl.n_requests,), 7, dtype=torch.uint8).pin_memory(),
                h_step_counters=torch.full((B.FB_STEP_COUNTERS,), -1, dtype=torch.int32).pin_memory(),
                h_status=torch.full((1,), -1, dtype=torch.int32).pin_memory(), n_rows=n_rows)
    B.fb_step_host(ctx2, st2, pk2, dev, host)
    torch.cuda.synchronize()
    assert int(host["h_status"][0]) == 0
    np.testing.assert_array_equal(host["h_n_committed"].numpy(), sb.n_committed.cpu().numpy())
    np.testing.assert_array_equal(host["h_spawned"].numpy(), sb.spawned.cpu().numpy())
    np.testing.assert_array_equal(host["h_step_counters"].numpy(), sb.step_counters.cpu().numpy())
    np.testing.assert_array_equal(sb2.out[:n_rows].float().cpu().numpy(), sb.out[:n_rows].float().cpu().numpy())
    a, b2 = st.to_numpy(), st2.to_numpy()
    for name in ("active", "prefix_len", "L", "R", "tokens", "pe_done"):
        np.testing.assert_array_equal(a[name], b2[name], err_msg=name)
    assert torch.equal(hkp, dkp) and torch.equal(hvp, dvp)
    assert bool((dev["logits"][n_rows:] == 0).all())      # rows beyond n_rows were not copied


# ------------------------------------- Eq. 6 as data movement (window in pages)
RESIDENT = ["tiny", "tiny_d128_b64", "tiny_wide", "tiny_noprefix", "tiny_b96", "tiny_g8", "cfg1"]


@pytest.mark.parametrize("name", RESIDENT)
@pytest.mark.parametrize("rope_base", [0.0, 10000.0])
def test_scatter_window_kv_and_resident_attention(name, rope_base):
    """fb_scatter_window_kv puts the fresh window K/V at their absolute
    positions (bit-exact without the rotary embedding, within bf16 rounding of
    the fp64 rotation with it) and touches nothing else; attention over the
    page-resident window matches the oracle; retirement then copies nothing."""
    case = make_case(WORKLOADS[name], with_logits=False)
    stc = case["stc"]
    wl = stc.wl
    b = wl.block_len
    ctx, st, pk, sb = gpu_objects(case, window_in_pages=1)
    q, kw, vw, kp, vp = case["attn"]
    dq, dkw, dvw, dkp, dvp = (t.to(DEV) for t in (q, kw, vw, kp, vp))
    B.fb_pack_wavefronts(ctx, st, pk, sb.ws, sb.status)
    B.fb_scatter_window_kv(ctx, pk, st.page_table, dkw, dvw, dkp, dvp, sb.status, rope_base=rope_base)
    sb.out.fill_(7.0)
    B.fb_wavefront_attn(ctx, pk, dq, None, None, dkp, dvp, st.page_table, sb.out, sb.ws, sb.status)
    torch.cuda.synchronize()
    assert int(sb.status.item()) == 0
    ocfg = H.oracle_cfg(stc)
    ost = H.oracle_state(stc, case["tokens"])
    opk = O.pack_wavefronts(ocfg, ost)
    check_pack(pk, opk)
    okp, ovp = H.f64(kp), H.f64(vp)
    O.scatter_window_kv(ocfg, opk, H.f64(kw), H.f64(vw), okp, ovp, stc.page_table, rope_base=rope_base)
    gk, gv = H.f64(dkp.cpu()), H.f64(dvp.cpu())
    np.testing.assert_array_equal(gv, ovp)
    if rope_base == 0.0:
        np.testing.assert_array_equal(gk, okp)
    else:
        # fp32 rotation of bf16 inputs, rounded to bf16: half an ulp of the result
        # (2^-9 relative) plus the fp32 arithmetic
        assert np.all(np.abs(gk - okp) <= 2.0 ** -8 * np.abs(okp) + 1e-6)
        untouched = okp == H.f64(kp)
        np.testing.assert_array_equal(gk[untouched], okp[untouched])
    # attention over what the GPU scattered (its own bf16 keys), against the oracle on the same pools
    ref = O.wavefront_attn(ocfg, opk, H.f64(q), None, None, gk, gv, stc.page_table)
    max_abs, rel = H.attn_errors(sb.out, ref, H.live_rows(opk, b))
    assert max_abs <= ATTN_MAX_ABS and rel <= ATTN_REL_L2, (max_abs, rel)
    assert bool((sb.out[opk.n_live * b:].float() == 7.0).all())
    # pointer-bump retirement: every block finished, pools stay as they are
    stats = torch.zeros_like(sb.slot_stats)
    toks = st.tokens.clone()
    toks[toks == stc.mask_id] = 1
    st.tokens.copy_(toks)
    ost.tokens[ost.tokens == stc.mask_id] = 1
    B.fb_gate_commit(ctx, pk, stats, st, None, None, None, None, sb.n_committed, sb.spawned,
                     sb.step_counters, sb.status)
    torch.cuda.synchronize()
    ncom, spawned, ctr = O.gate_commit(ocfg, opk, np.zeros((ocfg.max_slots, 6), np.int32), ost)
    np.testing.assert_array_equal(sb.n_committed.cpu().numpy(), ncom)
    g = st.to_numpy()
    for nm in ("active", "prefix_len", "L", "R"):
        np.testing.assert_array_equal(g[nm], getattr(ost, nm), err_msg=nm)
    assert torch.equal(dkp.cpu().view(torch.int16), torch.from_numpy(synth.to_bits(torch.from_numpy(gk).to(torch.bfloat16)).view(np.int16)).view(dkp.shape))


# ------------------------------------------------ degenerate and faulty inputs
def test_whole_step_on_an_empty_batch_touches_nothing():
    """No decoding request: every call is a no-op that leaves the outputs of
    padding rows, the state and the pools as they were."""
    wl = WORKLOADS["tiny"]
    case = make_case(wl)
    case["stc"].active[:] = 0
    stc = case["stc"]
    ctx, st, pk, sb = gpu_objects(case)
    q, kw, vw, kp, vp = (t.to(DEV) for t in case["attn"])
    kp0, vp0 = kp.clone(), vp.clone()
    z = case["logits"].to(DEV)
    before = st.to_numpy()
    sb.out.fill_(7.0)
    B.fb_pack_wavefronts(ctx, st, pk, sb.ws, sb.status)
    B.fb_wavefront_attn(ctx, pk, q, kw, vw, kp, vp, st.page_table, sb.out, sb.ws, sb.status)
    B.fb_t2t_step(ctx, pk, z, st, sb.argmax, sb.conf, sb.action, sb.slot_stats, sb.status)
    B.fb_gate_commit(ctx, pk, sb.slot_stats, st, kw, vw, kp, vp, sb.n_committed, sb.spawned,
                     sb.step_counters, sb.status)
    torch.cuda.synchronize()
    assert int(sb.status.item()) == 0 and int(pk.n_live.item()) == 0
    assert bool((sb.out.float() == 7.0).all())
    assert bool((sb.argmax == -1).all()) and bool((sb.conf == 0).all()) and bool((sb.action == 0).all())
    assert int(sb.slot_stats.abs().sum()) == 0 and int(sb.n_committed.abs().sum()) == 0
    assert int(sb.spawned.sum()) == 0
    after = st.to_numpy()
    for name in before:
        np.testing.assert_array_equal(after[name], before[name], err_msg=name)
    assert torch.equal(kp, kp0) and torch.equal(vp, vp0)


def test_faulty_inputs_set_status_bits_and_nothing_traps():
    """A page id outside the pool and a NaN logit are reported in the status
    word; the calls complete and the rows that are fine keep their parity."""
    wl = WORKLOADS["tiny"]
    case = make_case(wl)
    stc = case["stc"]
    r_bad = int(np.flatnonzero(stc.active == 1)[0])
    pt = stc.page_table.copy()
    pt[r_bad, 0] = stc.num_pages + 5                      # the first prefix page of one request
    ctx, st, pk, sb = gpu_objects(case)
    st.page_table.copy_(torch.from_numpy(pt))
    q, kw, vw, kp, vp = (t.to(DEV) for t in case["attn"])
    B.fb_pack_wavefronts(ctx, st, pk, sb.ws, sb.status)
    B.fb_wavefront_attn(ctx, pk, q, kw, vw, kp, vp, st.page_table, sb.out, sb.ws, sb.status)
    torch.cuda.synchronize()
    assert int(sb.status.item()) & B.FB_ST_BAD_PAGE
    # requests with intact page tables are unaffected
    ocfg = H.oracle_cfg(stc)
    opk = O.pack_wavefronts(ocfg, H.oracle_state(stc, case["tokens"]))
    good = [s for s in range(opk.n_live) if int(opk.slot_req[s]) != r_bad]
    ref = O.wavefront_attn(ocfg, opk, *(H.f64(t) for t in case["attn"]), stc.page_table, only_slots=good)
    max_abs, rel = H.attn_errors(sb.out, ref, H.live_rows(opk, wl.block_len, good))
    assert max_abs <= ATTN_MAX_ABS and rel <= ATTN_REL_L2
    # NaN logit in one live row
    sb.status.zero_()
    z = case["logits"].clone()
    z[3, 17] = float("nan")
    st2 = gpu_objects(case)[1]
    B.fb_t2t_step(ctx, pk, z.to(DEV), st2, sb.argmax, sb.conf, sb.action, sb.slot_stats, sb.status)
    torch.cuda.synchronize()
    assert int(sb.status.item()) & B.FB_ST_NAN_LOGIT
    assert float(sb.conf[3]) == 0.0 and int(sb.action[3]) == 0
    xhat, conf = O.t2t_rows(ocfg, opk, H.f64(case["logits"]))
    live = opk.n_live * wl.block_len
    keep = np.array([i for i in range(live) if i != 3])
    np.testing.assert_array_equal(sb.argmax.cpu().numpy()[keep], xhat[keep])
    np.testing.assert_allclose(sb.conf.cpu().numpy()[keep], conf[keep], rtol=0, atol=CONF_TOL)


@pytest.mark.parametrize("name", ["tiny", "tiny_wide", "cfg1"])
def test_embed_gather_bit_exact(name):
    case = make_case(WORKLOADS[name], with_attn=False, with_logits=False)
    stc = case["stc"]
    wl = stc.wl
    ctx, st, pk, sb = gpu_objects(case)
    hidden = 256
    table = synth.randn_bf16((wl.vocab, hidden), stc.seed, 12)
    x = torch.full((ctx.max_slots * wl.block_len, hidden), 7.0, dtype=torch.bfloat16, device=DEV)
    B.fb_pack_wavefronts(ctx, st, pk, sb.ws, sb.status)
    B.fb_embed_gather(ctx, pk, table.to(DEV), x, sb.status)
    torch.cuda.synchronize()
    assert int(sb.status.item()) == 0
    ocfg = H.oracle_cfg(stc)
    opk = O.pack_wavefronts(ocfg, H.oracle_state(stc, case["tokens"]))
    ref = O.embed_gather(ocfg, opk, H.f64(table))
    live = opk.n_live * wl.block_len
    np.testing.assert_array_equal(H.f64(x[:live].cpu()), ref[:live])
    assert bool((x[live:].float() == 7.0).all())
    # a table too short for the mask token is reported, nothing is read out of range
    B.fb_embed_gather(ctx, pk, table[:wl.vocab - 1].contiguous().to(DEV), x, sb.status)
    torch.cuda.synchronize()
    has_mask = bool((opk.qtok[:live] == stc.mask_id).any())
    assert bool(int(sb.status.item()) & B.FB_ST_BAD_TOKEN) == has_mask


# --------------------------------------------- LM head fused with the row pass
LM_TOL = 5e-5   # fp32 tensor-core accumulation of <= 256 bf16 products per logit against fp64: |dz| < 2e-5


WORKLOADS["tiny_v1000"] = synth.tiny_workload(vocab=1000, n_requests=5, w_lo=1, w_hi=3)   # ragged last vocabulary tile


@pytest.mark.parametrize("name,hidden", [("tiny", 128), ("tiny_wide", 64), ("tiny_d128_b64", 256),
                                         ("tiny_v1000", 192)])
def test_lm_head_fused_row_pass(name, hidden):
    """Top-1 token and confidence taken from x W^T on the tensor cores, the
    logits never written: winners bit-exact, confidences within the fp32
    accumulation error, then Eq. 1, the block counts and gate/commit exactly
    as with materialised logits."""
    case = make_case(WORKLOADS[name], with_attn=False, with_logits=False)
    stc = case["stc"]
    wl = stc.wl
    x, w, tokens = synth.make_lm_head_inputs(stc, case["tokens"], hidden)
    case["tokens"] = tokens
    ctx, st, pk, sb = gpu_objects(case)
    ws = torch.zeros(B.lib().fb_lm_head_workspace_bytes(ctx.handle), dtype=torch.uint8, device=DEV)
    B.fb_pack_wavefronts(ctx, st, pk, sb.ws, sb.status)
    B.fb_lm_head_t2t(ctx, pk, x.to(DEV), w.to(DEV), st, sb.argmax, sb.conf, sb.action, sb.slot_stats, ws,
                     sb.status)
    torch.cuda.synchronize()
    assert int(sb.status.item()) == 0
    ocfg = H.oracle_cfg(stc)
    ost = H.oracle_state(stc, tokens)
    opk = O.pack_wavefronts(ocfg, ost)
    xhat, conf = O.lm_head_rows(ocfg, opk, H.f64(x), H.f64(w))
    live = opk.n_live * wl.block_len
    for thr in (np.float32(ocfg.tau_mask), np.float32(ocfg.tau_edit)):
        assert np.abs(conf[:live] - float(thr)).min() >= MARGIN
    np.testing.assert_array_equal(sb.argmax.cpu().numpy(), xhat)
    np.testing.assert_allclose(sb.conf.cpu().numpy(), conf, rtol=0, atol=LM_TOL)
    action, stats = O.t2t_update(ocfg, opk, ost, xhat, conf)
    np.testing.assert_array_equal(sb.action.cpu().numpy(), action)
    np.testing.assert_array_equal(sb.slot_stats.cpu().numpy(), stats)
    np.testing.assert_array_equal(st.tokens.cpu().numpy(), ost.tokens)
    assert int((action == O.ACT_M2T).sum()) > 0


def test_step_host_with_the_window_in_pages():
    """fb_step_host in a window_in_pages context: scatter, attention over the
    pages, T2T, pointer-bump commit -- against the same calls made one by one."""
    wl = synth.tiny_workload(n_requests=4, prefix_lo=30, prefix_hi=260)
    case = make_case(wl, logits_kind="calibrated", conf_shift=0.25)
    stc = case["stc"]
    q, kw, vw, kp, vp = case["attn"]
    z = case["logits"]
    ctx, st, pk, sb = gpu_objects(case, window_in_pages=1)
    dq, dkw, dvw, dkp, dvp, dz = (t.to(DEV) for t in (q, kw, vw, kp, vp, z))
    B.fb_pack_wavefronts(ctx, st, pk, sb.ws, sb.status)
    B.fb_scatter_window_kv(ctx, pk, st.page_table, dkw, dvw, dkp, dvp, sb.status)
    B.fb_wavefront_attn(ctx, pk, dq, None, None, dkp, dvp, st.page_table, sb.out, sb.ws, sb.status)
    B.fb_t2t_step(ctx, pk, dz, st, sb.argmax, sb.conf, sb.action, sb.slot_stats, sb.status)
    B.fb_gate_commit(ctx, pk, sb.slot_stats, st, None, None, None, None, sb.n_committed, sb.spawned,
                     sb.step_counters, sb.status)
    torch.cuda.synchronize()
    assert int(sb.status.item()) == 0
    ctx2, st2, pk2, sb2 = gpu_objects(case, window_in_pages=1)
    n_rows = synth.n_live_slots(stc) * wl.block_len
    hkp, hvp = kp.to(DEV), vp.to(DEV)
    dev = dict(q=torch.zeros_like(dq), k_win=torch.zeros_like(dkw), v_win=torch.zeros_like(dvw), out=sb2.out,
               logits=torch.zeros_like(dz), k_pool=hkp, v_pool=hvp, argmax=sb2.argmax, conf=sb2.conf,
               action=sb2.action, slot_stats=sb2.slot_stats, n_committed=sb2.n_committed, spawned=sb2.spawned,
               step_counters=sb2.step_counters, status=sb2.status, ws=sb2.ws)
    host = dict(h_q=q.pin_memory(), h_k_win=kw.pin_memory(), h_v_win=vw.pin_memory(), h_logits=z.pin_memory(),
                h_n_committed=torch.full((wl.n_requests,), -1, dtype=torch.int32).pin_memory(),
                h_spawned=torch.full((wl.n_requests,), 7, dtype=torch.uint8).pin_memory(),
                h_step_counters=torch.full((B.FB_STEP_COUNTERS,), -1, dtype=torch.int32).pin_memory(),
                h_status=torch.full((1,), -1, dtype=torch.int32).pin_memory(), n_rows=n_rows)
    B.fb_step_host(ctx2, st2, pk2, dev, host)
    torch.cuda.synchronize()
    assert int(host["h_status"][0]) == 0
    np.testing.assert_array_equal(host["h_n_committed"].numpy(), sb.n_committed.cpu().numpy())
    np.testing.assert_array_equal(host["h_spawned"].numpy(), sb.spawned.cpu().numpy())
    np.testing.assert_array_equal(sb2.out[:n_rows].float().cpu().numpy(), sb.out[:n_rows].float().cpu().numpy())
    a, b2 = st.to_numpy(), st2.to_numpy()
    for name in ("active", "prefix_len", "L", "R", "tokens", "pe_done"):
        np.testing.assert_array_equal(a[name], b2[name], err_msg=name)
    assert torch.equal(hkp, dkp) and torch.equal(hvp, dvp)
    # and against the oracle: the committed prefix holds what the slot-order path would have copied
    ocfg = H.oracle_cfg(stc)
    ost = H.oracle_state(stc, case["tokens"])
    opk = O.pack_wavefronts(ocfg, ost)
    okp, ovp = H.f64(kp), H.f64(vp)
    ref = O.wavefront_attn(ocfg, opk, H.f64(q), H.f64(kw), H.f64(vw), okp, ovp, stc.page_table)
    max_abs, rel = H.attn_errors(sb2.out, ref, H.live_rows(opk, wl.block_len))
    assert max_abs <= ATTN_MAX_ABS and rel <= ATTN_REL_L2
    xhat, conf = O.t2t_rows(ocfg, opk, H.f64(z))
    action, stats = O.t2t_update(ocfg, opk, ost, xhat, conf)
    ncom, spawned, ctr = O.gate_commit(ocfg, opk, stats, ost, H.f64(kw), H.f64(vw), okp, ovp)
    np.testing.assert_array_equal(host["h_n_committed"].numpy(), ncom)
    ps = wl.page_size
    gk, gv = H.f64(hkp.cpu()), H.f64(hvp.cpu())
    for r in range(wl.n_requests):
        for pos in range(int(ost.prefix_len[r])):
            page, off = int(stc.page_table[r, pos // ps]), pos % ps
            np.testing.assert_array_equal(gk[page, :, off], okp[page, :, off])
            np.testing.assert_array_equal(gv[page, :, off], ovp[page, :, off])
