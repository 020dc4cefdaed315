"""CPU pins for the oracle's batch-synchronous wavefront (Sec. 3.2, first
paragraph; the packing ablation of Sec. 4.5): retirement gated by
``finished.all()``, admission by ``min_b rho_b``.

What the paper fixes: with one sequence the synchronous and the per-sequence
wavefront are the same thing (Sec. 4.5); a batch of identical sequences has no
straggler, so the two coincide there too; otherwise the slowest sequence holds
the others back.  The hand-worked cases spell that out on crafted block
counts.
"""
import dataclasses

import numpy as np
import pytest

from oracle import flowblock_oracle as O
from tests.test_oracle_t2t_gate import cfg4, step_logits_bank


def state(cfg, L, R, prefix=None, tokens=None):
    Rn, n, b = cfg.max_requests, cfg.max_blocks, cfg.block_len
    tok = np.full((Rn, n * b), cfg.mask_id, np.int32) if tokens is None else tokens
    return O.State(np.ones(Rn, np.int32),
                   np.zeros(Rn, np.int32) if prefix is None else np.array(prefix, np.int32),
                   np.array(L, np.int32), np.array(R, np.int32), tok,
                   np.zeros((Rn, cfg.wmax), np.uint8),
                   np.tile(np.arange(cfg.max_pages_per_req, dtype=np.int32), (Rn, 1)))


def slot_stats(cfg, pk, per_slot):
    """per_slot[(r, s)] = (m0, rdy, m2t, t2t, m1, eos); the rest: a block of
    four masks, none ready."""
    stats = np.zeros((cfg.max_slots, 6), np.int32)
    for i in range(pk.n_live):
        key = (int(pk.slot_req[i]), int(pk.slot_s[i]))
        stats[i] = per_slot.get(key, (4, 0, 0, 0, 4, 0))
    return stats


FIN = (0, 0, 0, 0, 0, 0)          # no masks, quiet forward: locally finished
FIN_EOS = (0, 0, 0, 0, 0, 1)
HALF = (4, 2, 0, 0, 4, 0)         # four masks, two of them ready: rho = 0.5
QUART = (4, 1, 0, 0, 4, 0)        # rho = 0.25


def both(cfg, st, per_slot):
    """(per-sequence result, synchronous result) from the same state."""
    out = []
    for mode in (0, 1):
        c = dataclasses.replace(cfg, batch_sync=mode)
        s = st.copy()
        pk = O.pack_wavefronts(c, s)
        res = O.gate_commit(c, pk, slot_stats(c, pk, per_slot), s)
        out.append((s, res))
    return out


def test_straggler_holds_retirement_back():
    cfg = cfg4(max_requests=2, wmax=2, max_blocks=6, s_pe=0)
    st = state(cfg, L=[0, 0], R=[2, 2])
    # request 0: oldest block finished; request 1: not
    (s0, (n0, sp0, c0)), (s1, (n1, sp1, c1)) = both(cfg, st, {(0, 0): FIN, (0, 1): HALF,
                                                                (1, 0): HALF, (1, 1): HALF})
    assert list(n0) == [1, 0] and list(s0.L) == [1, 0]
    assert list(n1) == [0, 0] and list(s1.L) == [0, 0] and list(s1.prefix_len) == [0, 0]
    assert c1[O.CT_LOCKSTEP_COMMIT] == 0 and c1[O.CT_BLOCKS] == 0
    # per sequence, request 0 now has room and rho = 0.5 >= theta: it admits; the batch cannot
    assert list(sp0) == [1, 0] and list(sp1) == [0, 0] and c1[O.CT_LOCKSTEP_ADMIT] == 0
    # both finished: both retire, and the cascade takes the second position only if both have it
    (_, _), (s1, (n1, sp1, c1)) = both(cfg, st, {(0, 0): FIN, (0, 1): FIN, (1, 0): FIN, (1, 1): HALF})
    assert list(n1) == [1, 1] and c1[O.CT_LOCKSTEP_COMMIT] == 1
    assert list(s1.L) == [1, 1] and list(s1.prefix_len) == [4, 4]
    # frontier rho: request 0 has no masks (1.0), request 1 has 0.5 -> min = 0.5 >= 0.5: all admit
    assert list(sp1) == [1, 1] and list(s1.R) == [3, 3] and c1[O.CT_LOCKSTEP_ADMIT] == 1
    assert c1[O.CT_SPAWNED] == 2 and c1[O.CT_TOKENS] == 8


def test_min_rho_gates_admission():
    cfg = cfg4(max_requests=3, wmax=3, max_blocks=6, theta_spawn=0.5)
    st = state(cfg, L=[0, 0, 0], R=[1, 1, 1])
    (s0, (_, sp0, _)), (s1, (_, sp1, c1)) = both(cfg, st, {(0, 0): HALF, (1, 0): QUART, (2, 0): HALF})
    assert list(sp0) == [1, 0, 1]                 # each sequence by its own rho
    assert list(sp1) == [0, 0, 0] and list(s1.R) == [1, 1, 1]   # min rho = 0.25 < 0.5
    (_, _), (s1, (_, sp1, c1)) = both(cfg, st, {(0, 0): HALF, (1, 0): HALF, (2, 0): HALF})
    assert list(sp1) == [1, 1, 1] and c1[O.CT_LOCKSTEP_ADMIT] == 1
    # the new blocks are all [M] and their post-edit counters start at 0
    assert (s1.tokens[:, 4:8] == cfg.mask_id).all() and (s1.pe_done == 0).all()
    # no room in one sequence (window full) -> nobody admits
    st = state(cfg, L=[0, 0, 0], R=[3, 1, 1])
    (_, _), (s1, (_, sp1, _)) = both(cfg, st, {(0, 0): HALF, (0, 1): HALF, (0, 2): HALF,
                                              (1, 0): HALF, (2, 0): HALF})
    assert list(sp1) == [0, 0, 0]


def test_committed_eos_leaves_the_batch_and_the_cascade_goes_on():
    cfg = cfg4(max_requests=2, wmax=2, max_blocks=6, s_pe=0, eos_id=3)
    st = state(cfg, L=[1, 1], R=[3, 3], prefix=[4, 4])
    (_, _), (s1, (n1, sp1, c1)) = both(cfg, st, {(0, 0): FIN_EOS, (0, 1): FIN, (1, 0): FIN, (1, 1): FIN})
    # position 0 retires in both; request 0 is done there; request 1 alone retires position 1
    assert list(n1) == [1, 2] and c1[O.CT_LOCKSTEP_COMMIT] == 2
    assert list(s1.active) == [2, 1] and c1[O.CT_FINISHED] == 1 and c1[O.CT_ACTIVE] == 1
    assert list(s1.L) == [2, 3] and list(s1.prefix_len) == [8, 12]
    assert list(sp1) == [0, 1]                    # the batch is request 1 now: empty window, rho = 1
    # an EOS behind a straggler's unfinished block is not committed: nobody leaves
    (_, _), (s1, (n1, _, c1)) = both(cfg, st, {(0, 0): FIN_EOS, (0, 1): FIN, (1, 0): HALF, (1, 1): FIN})
    assert list(n1) == [0, 0] and list(s1.active) == [1, 1]
    # a sequence that runs out of blocks (L reaches n) is done and does not block the others
    cfg = cfg4(max_requests=2, wmax=2, max_blocks=2, s_pe=0)
    st = state(cfg, L=[1, 0], R=[2, 2])
    (_, _), (s1, (n1, _, c1)) = both(cfg, st, {(0, 0): FIN, (1, 0): FIN, (1, 1): FIN})
    assert list(n1) == [1, 2] and list(s1.active) == [2, 2] and c1[O.CT_LOCKSTEP_COMMIT] == 2
    # handed in with L == n already: done at once under either policy, and no obstacle
    st = state(cfg, L=[2, 0], R=[2, 2])
    (s0, (n0, _, _)), (s1, (n1, _, c1)) = both(cfg, st, {(1, 0): FIN, (1, 1): HALF})
    assert list(n0) == list(n1) == [0, 1] and list(s0.active) == list(s1.active) == [2, 1]


def run(cfg, st, logits_for, steps):
    trace = []
    for step in range(steps):
        if not (st.active == 1).any():
            break
        pk = O.pack_wavefronts(cfg, st)
        *_, (ncom, sp, ctr) = O.decode_step(cfg, st, logits_for(cfg, st, pk, step))
        trace.append((ncom.copy(), sp.copy(), st.L.copy(), st.R.copy(), st.active.copy(), ctr.copy()))
    return trace


@pytest.mark.parametrize("seed,s_pe,W", [(1, 1, 3), (2, 0, 2), (3, 2, 4)])
def test_one_sequence_is_the_per_sequence_wavefront(seed, s_pe, W):
    """Sec. 4.5: at B = 1 the two implementations are semantically identical."""
    bl, n, V = 4, 6, 8
    bank = step_logits_bank(seed, 80, n, bl, V, forbid=[])
    bank[..., 7] -= 8.0                  # EOS rare but possible

    def logits_for(cfg, st, pk, step):
        z = np.zeros((cfg.max_slots * bl, V))
        for i in range(pk.n_live):
            z[i * bl:(i + 1) * bl] = bank[step, st.L[0] + pk.slot_s[i]]
        return z
    res = []
    for mode in (0, 1):
        cfg = cfg4(vocab=V, mask_id=8, eos_id=7, wmax=W, max_blocks=n, s_pe=s_pe, block_len=bl,
                   tau_mask=0.7, tau_edit=0.85, theta_spawn=0.4, batch_sync=mode)
        st = state(cfg, L=[0], R=[1])
        tr = run(cfg, st, logits_for, 80)
        res.append((tr, st))
    (ta, sa), (tb, sb) = res
    assert len(ta) == len(tb) and len(ta) > 3
    for x, y in zip(ta, tb):
        for u, v in zip(x[:5], y[:5]):
            np.testing.assert_array_equal(u, v)
        np.testing.assert_array_equal(x[5][:8], y[5][:8])       # the shared counters
    np.testing.assert_array_equal(sa.tokens, sb.tokens)
    assert sa.L[0] > 0


def test_identical_sequences_have_no_straggler():
    """Copies of one sequence: all() and min() over equal values change nothing."""
    bl, n, V, W, Rn = 4, 6, 8, 3, 3
    bank = step_logits_bank(21, 80, n, bl, V, forbid=[7])

    def logits_for(cfg, st, pk, step):
        z = np.zeros((cfg.max_slots * bl, V))
        for i in range(pk.n_live):
            z[i * bl:(i + 1) * bl] = bank[step, st.L[pk.slot_req[i]] + pk.slot_s[i]]
        return z
    res = []
    for mode in (0, 1):
        cfg = cfg4(max_requests=Rn, vocab=V, mask_id=8, eos_id=7, wmax=W, max_blocks=n, s_pe=1,
                   block_len=bl, tau_mask=0.7, tau_edit=0.85, theta_spawn=0.4, batch_sync=mode)
        st = state(cfg, L=[0] * Rn, R=[1] * Rn)
        res.append((run(cfg, st, logits_for, 80), st))
    (ta, sa), (tb, sb) = res
    assert len(ta) == len(tb)
    for x, y in zip(ta, tb):
        for u, v in zip(x[:5], y[:5]):
            np.testing.assert_array_equal(u, v)
    np.testing.assert_array_equal(sa.tokens, sb.tokens)
    assert (sa.L == n).all()


def test_lockstep_invariant_and_the_straggler_cost():
    """Different sequences from the same start: the synchronous windows stay
    equal at every step (the shared [L, R)), every block still commits in
    order, and no sequence is ever ahead of where its own wavefront would
    be (it waits for the slowest; it never skips a gate)."""
    bl, n, V, W, Rn = 4, 6, 8, 3, 4
    banks = [step_logits_bank(30 + r, 200, n, bl, V, forbid=[7]) for r in range(Rn)]

    def logits_for(cfg, st, pk, step):
        z = np.zeros((cfg.max_slots * bl, V))
        for i in range(pk.n_live):
            r = pk.slot_req[i]
            z[i * bl:(i + 1) * bl] = banks[r][step, st.L[r] + pk.slot_s[i]]
        return z
    out = {}
    for mode in (0, 1):
        cfg = cfg4(max_requests=Rn, vocab=V, mask_id=8, eos_id=7, wmax=W, max_blocks=n, s_pe=1,
                   block_len=bl, tau_mask=0.7, tau_edit=0.85, theta_spawn=0.4, batch_sync=mode)
        st = state(cfg, L=[0] * Rn, R=[1] * Rn)
        out[mode] = (run(cfg, st, logits_for, 200), st)
    tr, st = out[1]
    for ncom, sp, L, R, act, ctr in tr:
        live = act == 1
        if live.any():
            assert len(set(L[live])) == 1 and len(set(R[live])) == 1
        assert len(set(ncom)) == 1 and len(set(sp)) == 1      # nobody terminates early here (no EOS)
        assert ctr[O.CT_LOCKSTEP_COMMIT] == ncom[0] and ctr[O.CT_LOCKSTEP_ADMIT] == sp[0]
    assert (st.L == n).all() and (st.active == 2).all()
    # the per-sequence run finishes every sequence no later than the synchronous one
    steps_sync = len(out[1][0])
    done_at = [next(i for i, t in enumerate(out[0][0]) if t[4][r] == 2) for r in range(Rn)]
    assert max(done_at) + 1 <= steps_sync
    assert min(done_at) + 1 < steps_sync, "no straggler effect in this draw"
