"""CPU pins for the oracle's T2T step, readiness gate and in-order commit.

Closed forms, hand-worked Eq. 1 / Eq. 2 / Eq. 3 / Alg. 1 cases, and the
invariants "window of one block == serial block-wise decoding" (Sec. 2.2 /
3.1) and "packed == per-sequence execution" (Sec. 3.2).
"""
import math
import os

import numpy as np
import pytest

from oracle import flowblock_oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def cfg4(**kw):
    base = dict(max_requests=1, wmax=2, block_len=4, vocab=4, mask_id=4,
                eos_id=-1, max_blocks=4, s_pe=1, tau_mask=0.9, tau_edit=0.95,
                theta_spawn=0.5, page_size=4, num_pages=16,
                max_pages_per_req=8)
    base.update(kw)
    return O.Config(**base)


def one_request_state(cfg, tokens_live, L=0, R=1, prefix=0):
    n, b = cfg.max_blocks, cfg.block_len
    tok = np.full((cfg.max_requests, n * b), cfg.mask_id, np.int32)
    tok[0, L * b:L * b + len(tokens_live)] = tokens_live
    return O.State(np.array([1] + [0] * (cfg.max_requests - 1), np.int32),
                   np.array([prefix] * cfg.max_requests, np.int32),
                   np.array([L] * cfg.max_requests, np.int32),
                   np.array([R] * cfg.max_requests, np.int32), tok,
                   np.zeros((cfg.max_requests, cfg.wmax), np.uint8),
                   np.tile(np.arange(cfg.max_pages_per_req, dtype=np.int32),
                           (cfg.max_requests, 1)))


def peaked_rows(V, spec):
    """rows 'one logit = a, the others 0'; spec = [(winner, a), ...]"""
    z = np.zeros((len(spec), V))
    for i, (w, a) in enumerate(spec):
        z[i, w] = a
    return z


# ----------------------------------------------------------- confidence
@pytest.mark.parametrize("a,expect", [(0, 0.25), (2, 0.71123), (3, 0.87005),
                                      (4, 0.94791), (5, 0.98019),
                                      (6, 0.99262)])
def test_confidence_closed_form_V4(a, expect):
    cfg = cfg4()
    st = one_request_state(cfg, [4, 4, 4, 4])
    pk = O.pack_wavefronts(cfg, st)
    z = np.zeros((cfg.max_slots * 4, 4))
    z[:4] = peaked_rows(4, [(2, a)] * 4)
    xhat, conf = O.t2t_rows(cfg, pk, z)
    # p = e^a / (e^a + V - 1), value also quoted to 5 decimals
    assert abs(conf[0] - math.exp(a) / (math.exp(a) + 3)) < 1e-15
    assert abs(conf[0] - expect) < 6e-6
    assert xhat[0] == (2 if a > 0 else 0)       # 4-way tie -> lowest index
    assert xhat[4] == -1 and conf[4] == 0.0     # padding slot


def test_confidence_large_vocab_and_ties():
    V = 151552
    cfg = cfg4(vocab=V, mask_id=V - 1)
    st = one_request_state(cfg, [V - 1] * 4)
    pk = O.pack_wavefronts(cfg, st)
    z = np.zeros((cfg.max_slots * 4, V))
    z[0, 777] = 13.0
    z[1, [5, 900, 151000]] = 3.0                # three-way tie
    z[2] = -4.0; z[2, V - 1] = -4.0             # all equal
    z[3, 12345] = 20.0; z[3, 2] = 19.0
    xhat, conf = O.t2t_rows(cfg, pk, z)
    assert xhat[0] == 777
    assert abs(conf[0] - 1 / (1 + (V - 1) * math.exp(-13.0))) < 1e-14
    assert xhat[1] == 5
    assert abs(conf[1] - 1 / (3 + (V - 3) * math.exp(-3.0))) < 1e-14
    assert xhat[2] == 0 and abs(conf[2] - 1 / V) < 1e-18
    assert xhat[3] == 12345
    assert abs(conf[3] - 1 / (1 + math.exp(-1) + (V - 2) * math.exp(-20))) < 1e-14


# ------------------------------------------------- hand-worked Eq.1/2/3
def worked_case(theta=0.5, wmax=2, R=1, n=4):
    cfg = cfg4(theta_spawn=theta, wmax=wmax, max_blocks=n)
    st = one_request_state(cfg, [4, 4, 3, 0], L=0, R=R)
    pk = O.pack_wavefronts(cfg, st)
    z = np.zeros((cfg.max_slots * 4, 4))
    z[:4] = peaked_rows(4, [(2, 5), (1, 3), (1, 5), (3, 4)])
    return cfg, st, pk, z


def test_hand_worked_update_and_gate():
    cfg, st, pk, z = worked_case()
    xhat, conf = O.t2t_rows(cfg, pk, z)
    np.testing.assert_allclose(conf[:4], [0.98019, 0.87005, 0.98019, 0.94791],
                               atol=6e-6)
    action, stats = O.t2t_update(cfg, pk, st, xhat, conf)
    # pos0 [M] -> 2 (M2T); pos1 stays [M] (.870 <= .9); pos2 3 -> 1 (T2T);
    # pos3 not edited (.948 <= .95)
    assert list(st.tokens[0, :4]) == [2, 4, 1, 0]
    assert list(action[:4]) == [O.ACT_M2T, O.ACT_NONE, O.ACT_T2T, O.ACT_NONE]
    assert list(stats[0]) == [2, 1, 1, 1, 1, 0]    # m0 rdy m2t t2t m1 eos
    ncom, spawned, ctr = O.gate_commit(cfg, pk, stats, st)
    # not finished (a mask remains); rho = 1/2 >= .5 -> admit block 1
    assert ncom[0] == 0 and spawned[0] == 1
    assert (st.L[0], st.R[0], st.prefix_len[0]) == (0, 2, 0)
    assert (st.tokens[0, 4:8] == cfg.mask_id).all()
    assert ctr[O.CT_SPAWNED] == 1 and ctr[O.CT_M2T] == 1 and ctr[O.CT_T2T] == 1


def test_gate_variants():
    # theta just above 1/2 -> no admission
    cfg, st, pk, z = worked_case(theta=0.51)
    xh, cf = O.t2t_rows(cfg, pk, z)
    _, stats = O.t2t_update(cfg, pk, st, xh, cf)
    _, spawned, _ = O.gate_commit(cfg, pk, stats, st)
    assert spawned[0] == 0 and st.R[0] == 1
    # window already full (R - L == W) -> no admission
    cfg, st, pk, z = worked_case(wmax=1)
    xh, cf = O.t2t_rows(cfg, pk, z)
    _, stats = O.t2t_update(cfg, pk, st, xh, cf)
    _, spawned, _ = O.gate_commit(cfg, pk, stats, st)
    assert spawned[0] == 0
    # no block left (R == n) -> no admission
    cfg, st, pk, z = worked_case(n=1)
    xh, cf = O.t2t_rows(cfg, pk, z)
    _, stats = O.t2t_update(cfg, pk, st, xh, cf)
    _, spawned, _ = O.gate_commit(cfg, pk, stats, st)
    assert spawned[0] == 0


def test_admission_table_binary32():
    for line in open(os.path.join(GOLD, "admission_equality.txt")):
        if line.startswith("#") or not line.strip():
            continue
        rdy, m0, theta, admit = line.split()
        cfg = cfg4(theta_spawn=float(theta), s_pe=5)
        toks = [4] * int(m0) + [1] * (4 - min(4, int(m0)))
        st = one_request_state(cfg, toks[:4])
        pk = O.pack_wavefronts(cfg, st)
        stats = np.zeros((cfg.max_slots, 6), np.int32)
        stats[0] = [int(m0), int(rdy), 0, 0, max(1, int(m0)), 0]
        _, spawned, _ = O.gate_commit(cfg, pk, stats, st)
        assert spawned[0] == int(admit), line


def test_strict_and_nonstrict_thresholds():
    """Eq. 1 reveals on p > tau_mask, Eq. 2 counts p >= tau_mask."""
    cfg = cfg4(tau_mask=0.5, tau_edit=0.5)       # exactly representable
    st = one_request_state(cfg, [4, 4, 1, 1])
    pk = O.pack_wavefronts(cfg, st)
    xhat = np.array([2, 2, 2, 2] + [-1] * 4, np.int32)
    conf = np.array([0.5, 0.5000001, 0.5, 0.5000001] + [0] * 4)
    action, stats = O.t2t_update(cfg, pk, st, xhat, conf)
    assert list(action[:4]) == [0, O.ACT_M2T, 0, O.ACT_T2T]
    assert stats[0, O.ST_RDY] == 2 and stats[0, O.ST_M2T] == 1


# ----------------------------------------------------- commit behaviour
def run_steps(cfg, st, logits_fn, steps, kv=None):
    trace = []
    for t in range(steps):
        if not (st.active == 1).any():
            break
        pk = O.pack_wavefronts(cfg, st)
        z = logits_fn(t, pk, st)
        _, xh, cf, act, stats, (ncom, sp, ctr) = O.decode_step(cfg, st, z, kv)
        trace.append((t, ncom.copy(), sp.copy(), ctr.copy()))
    return trace


def test_finish_needs_a_quiet_step_or_spe_budget():
    V = 4
    # all revealed, model agrees -> no update -> finished at once (early stop)
    cfg = cfg4(s_pe=3)
    st = one_request_state(cfg, [1, 1, 1, 1])
    pk = O.pack_wavefronts(cfg, st)
    z = np.zeros((8, V)); z[:4, 1] = 6
    *_, (ncom, sp, ctr) = O.decode_step(cfg, st, z)
    assert ncom[0] == 1 and st.L[0] == 1 and st.prefix_len[0] == 4
    assert sp[0] == 1 and st.R[0] == 2          # empty window -> rho = 1
    # edits keep coming: block is held for exactly S_pe post-edit forwards
    for s_pe in (0, 1, 3):
        cfg = cfg4(s_pe=s_pe, wmax=1)
        st = one_request_state(cfg, [4, 4, 4, 4])
        commits = []
        for step in range(8):
            pk = O.pack_wavefronts(cfg, st)
            if st.L[0] > 0:
                break
            z = np.zeros((4, V)); z[:, step % 3] = 6  # winner changes / step
            *_, (ncom, sp, ctr) = O.decode_step(cfg, st, z)
            commits.append(int(ncom[0]))
        # step 0 reveals all masks; then S_pe further forwards, each editing
        assert commits.index(1) == s_pe, (s_pe, commits)


def test_cascade_and_eos_stop():
    V = 6
    cfg = cfg4(vocab=V, mask_id=6, eos_id=5, wmax=3, max_blocks=6, s_pe=0)
    # three live blocks, all fully revealed and stable -> all three retire
    st = one_request_state(cfg, [1] * 12, L=1, R=4, prefix=8)
    z = np.zeros((12, V)); z[:, 1] = 7
    *_, (ncom, sp, ctr) = O.decode_step(cfg, st, z)
    assert ncom[0] == 3 and st.L[0] == 4 and st.prefix_len[0] == 8 + 12
    assert sp[0] == 1 and st.R[0] == 5 and ctr[O.CT_TOKENS] == 12
    # middle block unfinished -> only the first retires (in-order)
    st = one_request_state(cfg, [1] * 4 + [6, 1, 1, 1] + [1] * 4, L=1, R=4)
    z = np.zeros((12, V)); z[:, 1] = 7; z[4] = 0
    *_, (ncom, sp, ctr) = O.decode_step(cfg, st, z)
    assert ncom[0] == 1 and st.L[0] == 2
    # the frontier block has no masks (rho = 1) and the window now has room
    assert sp[0] == 1 and st.R[0] == 5
    # EOS inside the second block: cascade stops there, request is done, the
    # third (finished) block is dropped
    st = one_request_state(cfg, [1] * 4 + [1, 5, 1, 1] + [1] * 4, L=1, R=4)
    z = np.zeros((12, V)); z[:, 1] = 7; z[5] = 0; z[5, 5] = 7
    *_, (ncom, sp, ctr) = O.decode_step(cfg, st, z)
    assert ncom[0] == 2 and st.active[0] == 2 and sp[0] == 0
    assert ctr[O.CT_FINISHED] == 1
    # an EOS in a block that cannot commit yet does not terminate
    st = one_request_state(cfg, [6, 1, 1, 1] + [1, 5, 1, 1], L=0, R=2)
    z = np.zeros((12, V)); z[:, 1] = 7; z[0] = 0; z[5] = 0; z[5, 5] = 7
    *_, (ncom, sp, ctr) = O.decode_step(cfg, st, z)
    assert ncom[0] == 0 and st.active[0] == 1
    # last block committed -> done even without EOS
    cfg = cfg4(vocab=V, mask_id=6, eos_id=5, wmax=2, max_blocks=2, s_pe=0)
    st = one_request_state(cfg, [1] * 4, L=1, R=2)
    z = np.zeros((8, V)); z[:, 1] = 7
    *_, (ncom, sp, ctr) = O.decode_step(cfg, st, z)
    assert st.L[0] == 2 and st.active[0] == 2


def test_commit_freezes_kv_and_never_touches_older_pages():
    rng = np.random.default_rng(2)
    cfg = cfg4(vocab=6, mask_id=6, wmax=2, max_blocks=6, s_pe=2, n_kv_heads=2,
               n_q_heads=2, head_dim=8, num_pages=16, max_pages_per_req=8)
    st = one_request_state(cfg, [1] * 8, L=1, R=3, prefix=6)  # unaligned
    st.page_table[0] = rng.permutation(16)[:8]
    kw = rng.standard_normal((cfg.max_slots * 4, 2, 8))
    vw = rng.standard_normal((cfg.max_slots * 4, 2, 8))
    kp = rng.standard_normal((16, 2, 4, 8)); vp = rng.standard_normal((16, 2, 4, 8))
    kp0, vp0 = kp.copy(), vp.copy()
    z = np.zeros((8, 6)); z[:4, 1] = 7; z[4:, 2] = 9  # block 2 still editing
    *_, (ncom, sp, ctr) = O.decode_step(cfg, st, z, (kw, vw, kp, vp))
    assert ncom[0] == 1
    changed = set()
    for j in range(6, 10):                           # absolute positions
        pg = st.page_table[0, j // 4]
        np.testing.assert_array_equal(kp[pg, :, j % 4], kw[j - 6])
        np.testing.assert_array_equal(vp[pg, :, j % 4], vw[j - 6])
        changed.add((pg, j % 4))
    for pg in range(16):
        for o in range(4):
            if (pg, o) not in changed:
                np.testing.assert_array_equal(kp[pg, :, o], kp0[pg, :, o])
                np.testing.assert_array_equal(vp[pg, :, o], vp0[pg, :, o])


# ---------------------------------------- W = 1  ==  serial block-wise
def step_logits_bank(seed, steps, n_blocks, bl, V, forbid):
    rng = np.random.default_rng(seed)
    z = rng.standard_normal((steps, n_blocks, bl, V))
    win = rng.integers(0, V - len(forbid), size=(steps, n_blocks, bl))
    boost = rng.choice([0.0, 4.0, 6.5, 9.0], size=(steps, n_blocks, bl))
    for idx in np.ndindex(steps, n_blocks, bl):
        z[idx][win[idx]] += boost[idx]
    for f in forbid:
        z[..., f] = -30.0
    return z


@pytest.mark.parametrize("s_pe,seed", [(0, 1), (1, 2), (1, 3), (3, 4)])
def test_window_of_one_equals_serial_decoder(s_pe, seed):
    bl, n, V = 4, 5, 8
    cfg = cfg4(vocab=V, mask_id=8, eos_id=7, wmax=1, max_blocks=n, s_pe=s_pe,
               block_len=bl, tau_mask=0.6, tau_edit=0.8)
    bank = step_logits_bank(seed, 200, n, bl, V, forbid=[])
    bank[..., 7] -= 3.0                  # EOS rare but possible
    ser_tok, events, used = O.serial_blockwise_decode(
        bl, n, cfg.mask_id, cfg.eos_id, cfg.tau_mask, cfg.tau_edit, s_pe,
        lambda step, blk: bank[step, blk])
    st = one_request_state(cfg, [cfg.mask_id] * bl)
    got_events = []
    for step in range(200):
        if st.active[0] != 1:
            break
        blk = int(st.L[0])
        z = np.zeros((cfg.max_slots * bl, V)); z[:bl] = bank[step, blk]
        *_, (ncom, sp, ctr) = O.decode_step(cfg, st, z)
        if ncom[0]:
            got_events.append((step, blk))
    assert got_events == events and len(events) >= 1
    ncommitted = len(events) * bl
    np.testing.assert_array_equal(st.tokens[0, :ncommitted],
                                  ser_tok[:ncommitted])


# ------------------------------------ packed  ==  per-sequence execution
def test_packed_equals_independent_requests():
    bl, n, V, W, Rn = 4, 6, 8, 3, 4
    banks = [step_logits_bank(10 + r, 60, n, bl, V, forbid=[7]) for r in range(Rn)]
    def make(Rmax):
        return cfg4(max_requests=Rmax, vocab=V, mask_id=8, eos_id=7, wmax=W,
                    max_blocks=n, s_pe=1, block_len=bl, tau_mask=0.7,
                    tau_edit=0.85, theta_spawn=0.4)
    def logits_for(cfg, st, pk, step, req_ids):
        z = np.zeros((cfg.max_slots * bl, V))
        for i in range(pk.n_live):
            r = pk.slot_req[i]
            g = st.L[r] + pk.slot_s[i]
            z[i * bl:(i + 1) * bl] = banks[req_ids[r]][step, g]
        return z
    # together
    cfg = make(Rn)
    st = O.State(np.ones(Rn, np.int32), np.array([3, 0, 9, 5], np.int32),
                 np.zeros(Rn, np.int32), np.ones(Rn, np.int32),
                 np.full((Rn, n * bl), 8, np.int32), np.zeros((Rn, W), np.uint8),
                 np.zeros((Rn, 8), np.int32))
    tog = []
    for step in range(60):
        pk = O.pack_wavefronts(cfg, st)
        z = logits_for(cfg, st, pk, step, list(range(Rn)))
        *_, (ncom, sp, ctr) = O.decode_step(cfg, st, z)
        tog.append((ncom.copy(), sp.copy(), st.L.copy(), st.R.copy()))
    # one by one
    for r in range(Rn):
        c1 = make(1)
        s1 = O.State(np.ones(1, np.int32), np.array([[3, 0, 9, 5][r]], np.int32),
                     np.zeros(1, np.int32), np.ones(1, np.int32),
                     np.full((1, n * bl), 8, np.int32), np.zeros((1, W), np.uint8),
                     np.zeros((1, 8), np.int32))
        for step in range(60):
            pk = O.pack_wavefronts(c1, s1)
            z = logits_for(c1, s1, pk, step, [r])
            *_, (ncom, sp, ctr) = O.decode_step(c1, s1, z)
            assert ncom[0] == tog[step][0][r] and sp[0] == tog[step][1][r]
            assert s1.L[0] == tog[step][2][r] and s1.R[0] == tog[step][3][r]
        np.testing.assert_array_equal(s1.tokens[0], st.tokens[r])
        assert s1.active[0] == st.active[r]
    assert (st.L > 0).all()          # the run actually committed blocks
