"""Serving sweep on the GPU against the oracle, state by state: 128 requests
arriving over 24 steps, 48 steps in all, confidences rising by 0.05 per step
(the serving workload's structure: 512 slots, 64 blocks per request, prefixes of
512-4096 tokens; the vocabulary is cut to 4096 so that the oracle's own row
pass over every live row of every step stays affordable).  After every step the tokens, the
window bounds, the prefix lengths, the per-step outputs and the frozen K/V of
the blocks that retired are compared; commits and admissions of one step feed
the next one on both sides."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import flowblock_oracle as O
from paper_2607_17652_b200 import sweep, synth
from tests import harness as H

pytestmark = pytest.mark.gpu
CONF_TOL = 2e-5


def _frozen_kv_matches(run, opk, ost_before, ncom, b):
    """Pool rows [P_old, P_old + c*bl) of every request that retired c blocks
    equal the window K/V rows of those blocks, byte for byte (Eq. 6)."""
    kp, vp, kw, vw = run.kp, run.vp, run.kw, run.vw
    pt = ost_before.page_table
    for r in np.flatnonzero(ncom > 0):
        P0 = int(ost_before.prefix_len[r])
        slot0 = int(opk.req_slot_begin[r])
        n = int(ncom[r]) * b
        pos = np.arange(P0, P0 + n)
        pages = torch.from_numpy(pt[r, pos // 64].astype(np.int64)).to(kp.device)
        offs = torch.from_numpy((pos % 64).astype(np.int64)).to(kp.device)
        rows = torch.arange(slot0 * b, slot0 * b + n, device=kp.device)
        if not (torch.equal(kp[pages, :, offs], kw[rows]) and torch.equal(vp[pages, :, offs], vw[rows])):
            return False
    return True


@pytest.mark.parametrize("window_in_pages,batch_sync", [(False, False), (True, False), (False, True)])
def test_serving_sweep_states_match_oracle_every_step(window_in_pages, batch_sync):
    """window_in_pages: the same sequence with the window K/V scattered into the
    pages every step (Eq. 6) and retirement as a pointer bump; the frozen K/V
    must come out the same.  batch_sync: the batch-synchronous wavefront of the
    packing ablation on a static batch (every request there at step 0)."""
    wl = dataclasses.replace(synth.WORKLOADS[4], vocab=4096)
    n_steps = 48
    # EOS winners from the third block on, so that some requests terminate within the 48 steps
    inp = sweep.SweepInputs(wl, n_steps=n_steps, eos_min_block=2, arrive_hi=1 if batch_sync else 24)
    run = sweep.SweepRunner(inp, window_in_pages=window_in_pages, batch_sync=batch_sync)
    stc = inp.stc
    b = wl.block_len
    ocfg = H.oracle_cfg(stc, batch_sync=int(batch_sync))
    ost = H.oracle_state(stc, inp.tokens0())
    n_rows = wl.max_slots * b
    commits = spawns = edits = 0
    for step in range(n_steps):
        for r in inp.arrivals(step):                      # the caller writes the state row
            ost.active[r] = 1
            run.arrive(r)
        rows, cols, vals, conf = inp.begin_step(step, ost.active, ost.L, ost.R)
        inp.apply(run.z, rows, cols, vals)
        run.step()
        sb = run.sb
        assert int(sb.status.item()) == 0
        opk = O.pack_wavefronts(ocfg, ost)
        g = run.pk.to_numpy()
        assert int(g["n_live"][0]) == opk.n_live == len(rows) // b
        for name in ("slot_req", "slot_s", "slot_pos0", "slot_kv_len", "slot_flags", "req_slot_begin",
                     "qtok", "pos"):
            np.testing.assert_array_equal(g[name], getattr(opk, name), err_msg=f"{name}@{step}")
        # Expected winners and confidences of EVERY step come from the oracle's own plain row
        # pass over the patched logits as they stand on the device; the values the input
        # generator declares for its patches are only cross-checked against them.
        full = np.zeros((n_rows, wl.vocab))
        full[:len(rows)] = H.f64(run.z[:len(rows)].cpu())
        xhat, cf = O.t2t_rows(ocfg, opk, full)
        np.testing.assert_array_equal(xhat[:len(rows)], cols, err_msg=f"declared winners@{step}")
        assert np.abs(cf[:len(rows)] - conf).max() < 1e-12, f"declared confidences@{step}"
        before = dataclasses.replace(ost, prefix_len=ost.prefix_len.copy())
        action, stats = O.t2t_update(ocfg, opk, ost, xhat, cf)
        ncom, spawned, ctr = O.gate_commit(ocfg, opk, stats, ost)
        live = slice(0, len(rows))
        np.testing.assert_array_equal(sb.argmax.cpu().numpy()[live], xhat[live])
        assert np.abs(sb.conf.cpu().numpy()[live].astype(np.float64) - cf[live]).max() <= CONF_TOL
        np.testing.assert_array_equal(sb.action.cpu().numpy(), action)
        np.testing.assert_array_equal(sb.slot_stats.cpu().numpy()[:opk.n_live], stats[:opk.n_live])
        np.testing.assert_array_equal(sb.n_committed.cpu().numpy(), ncom)
        np.testing.assert_array_equal(sb.spawned.cpu().numpy(), spawned)
        np.testing.assert_array_equal(sb.step_counters.cpu().numpy(), ctr)
        gs = run.st.to_numpy()
        for name in ("active", "prefix_len", "L", "R", "tokens", "pe_done"):
            np.testing.assert_array_equal(gs[name], getattr(ost, name), err_msg=f"{name}@{step}")
        assert _frozen_kv_matches(run, opk, before, ncom, b), f"frozen K/V @ {step}"
        commits += int(ncom.sum())
        spawns += int(spawned.sum())
        edits += int((action == O.ACT_T2T).sum())
    assert (ost.active != 0).all(), "every request has arrived"
    assert edits > 0, "the re-drawn winners never produced a T2T edit"
    if batch_sync:
        # the shared window: every sequence still decoding sits at the same [L, R)
        live = ost.active == 1
        assert len(set(ost.L[live])) <= 1 and len(set(ost.R[live])) <= 1
        assert commits >= wl.n_requests
    else:
        assert commits >= 2 * wl.n_requests and spawns >= commits
        assert (ost.active == 2).any(), "no request reached a committed EOS"
