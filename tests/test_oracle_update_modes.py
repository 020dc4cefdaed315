"""CPU pins for the two optional modes of the oracle's Eq. 1 update: Delta taken
literally (masked positions too) and the forced-progress rule on the oldest
block.  Hand-worked rows with the closed-form confidences
p = e^a / (e^a + V - 1), the cases where a mode must change nothing, and the
termination bound the forced rule exists for.
"""
import dataclasses

import numpy as np
import pytest

from oracle import flowblock_oracle as O
from tests.test_oracle_t2t_gate import cfg4, one_request_state, peaked_rows, step_logits_bank


def update(cfg, tokens_live, spec, R=1, n_live_blocks=1):
    st = one_request_state(cfg, tokens_live, L=0, R=R)
    pk = O.pack_wavefronts(cfg, st)
    z = np.zeros((cfg.max_slots * cfg.block_len, cfg.vocab))
    z[:len(spec)] = peaked_rows(cfg.vocab, spec)
    xhat, conf = O.t2t_rows(cfg, pk, z)
    action, stats = O.t2t_update(cfg, pk, st, xhat, conf)
    return st, action, stats, conf


def test_literal_delta_hand_worked():
    # V = 4: a = 3 -> p = .87005, a = 4 -> .94791, a = 5 -> .98019
    # thresholds the "wrong way round": tau_edit = .85 < tau_mask = .96
    spec = [(2, 3), (1, 4), (1, 5), (3, 2)]
    toks = [4, 4, 3, 4]                       # [M] [M] token3 [M]
    base = cfg4(tau_mask=0.96, tau_edit=0.85)
    # revealed-only Delta (default reading): only p > .96 reveals a mask; the revealed
    # position 2 (3 -> 1, p = .980 > .85) is edited
    st, act, stats, conf = update(base, toks, spec)
    assert list(st.tokens[0, :4]) == [4, 4, 1, 4]
    assert list(act[:4]) == [0, 0, O.ACT_T2T, 0] and list(stats[0]) == [3, 0, 0, 1, 3, 0]
    # literal Delta: masks with p > tau_edit are updated too (.870 and .948 > .85; .711 is not)
    lit = dataclasses.replace(base, delta_literal=1)
    st, act, stats, conf = update(lit, toks, spec)
    assert list(st.tokens[0, :4]) == [2, 1, 1, 4]
    assert list(act[:4]) == [O.ACT_M2T, O.ACT_M2T, O.ACT_T2T, 0]
    # Eq. 2 still counts readiness against tau_mask: none of the three masks had p >= .96
    assert list(stats[0]) == [3, 0, 2, 1, 1, 0]
    # a mask whose own prediction is [M] is not in Delta (x != x_hat fails): mask_id inside the vocabulary
    cfgm = cfg4(vocab=4, mask_id=3, tau_mask=0.96, tau_edit=0.85, delta_literal=1)
    st, act, stats, _ = update(cfgm, [3, 3, 0, 0], [(3, 4), (1, 4), (0, 5), (0, 5)])
    assert list(st.tokens[0, :4]) == [3, 1, 0, 0] and list(act[:4]) == [0, O.ACT_M2T, 0, 0]


@pytest.mark.parametrize("seed", range(4))
def test_literal_delta_changes_nothing_when_tau_edit_is_not_below_tau_mask(seed):
    """Sec. 2.1's thresholds in their usual order: every masked position in the
    literal Delta is in Gamma already."""
    bl, n, V = 4, 5, 8
    bank = step_logits_bank(40 + seed, 60, n, bl, V, forbid=[7])
    res = []
    for lit in (0, 1):
        cfg = cfg4(vocab=V, mask_id=8, eos_id=7, wmax=3, max_blocks=n, s_pe=1, block_len=bl,
                   tau_mask=0.7, tau_edit=0.7 + 0.1 * (seed % 2), theta_spawn=0.4, delta_literal=lit)
        st = one_request_state(cfg, [8] * bl)
        trace = []
        for step in range(60):
            if st.active[0] != 1:
                break
            pk = O.pack_wavefronts(cfg, st)
            z = np.zeros((cfg.max_slots * bl, V))
            for i in range(pk.n_live):
                z[i * bl:(i + 1) * bl] = bank[step, st.L[0] + pk.slot_s[i]]
            _, xh, cf, act, stats, (ncom, sp, ctr) = O.decode_step(cfg, st, z)
            trace.append((act.copy(), stats.copy(), int(ncom[0]), int(sp[0])))
        res.append((trace, st.tokens.copy()))
    assert len(res[0][0]) == len(res[1][0])
    for a, b in zip(res[0][0], res[1][0]):
        np.testing.assert_array_equal(a[0], b[0]); np.testing.assert_array_equal(a[1], b[1])
        assert a[2:] == b[2:]
    np.testing.assert_array_equal(res[0][1], res[1][1])


def test_forced_progress_hand_worked():
    # two live blocks, nothing clears tau_mask = .9 anywhere: p = .711, .870, .870, .500 / .870 x4
    cfg = cfg4(force_progress=1, wmax=2)
    spec = [(2, 2), (1, 3), (3, 3), (0, 1.0986122886681098)] + [(1, 3)] * 4
    st, act, stats, conf = update(cfg, [4, 4, 4, 0] + [4] * 4, spec, R=2)
    np.testing.assert_allclose(conf[:4], [0.71123, 0.87005, 0.87005, 0.5], atol=6e-6)
    # oldest block: the best masked position is 1 (tie with 2 -> lower position); position 3 is
    # revealed already and does not compete.  The younger block is left alone.
    assert list(st.tokens[0, :8]) == [4, 1, 4, 0, 4, 4, 4, 4]
    assert list(act[:8]) == [0, O.ACT_FORCED, 0, 0, 0, 0, 0, 0]
    assert list(stats[0]) == [3, 0, 1, 0, 2, 0] and list(stats[1]) == [4, 0, 0, 0, 4, 0]
    # the same block without the rule: nothing happens
    st, act, stats, _ = update(cfg4(wmax=2), [4, 4, 4, 0] + [4] * 4, spec, R=2)
    assert not act.any() and list(stats[0]) == [3, 0, 0, 0, 3, 0]
    # Eq. 1 reveals something in the oldest block -> the rule stays out of it
    spec2 = [(2, 5)] + spec[1:]
    st, act, stats, _ = update(cfg, [4, 4, 4, 0] + [4] * 4, spec2, R=2)
    assert list(act[:4]) == [O.ACT_M2T, 0, 0, 0] and list(stats[0]) == [3, 1, 1, 0, 2, 0]
    # an edit is not a reveal: the rule still fires beside it
    spec3 = [(2, 2), (1, 3), (3, 3), (1, 5)] + [(1, 3)] * 4
    st, act, stats, _ = update(cfg, [4, 4, 4, 0] + [4] * 4, spec3, R=2)
    assert list(act[:4]) == [0, O.ACT_FORCED, 0, O.ACT_T2T] and list(stats[0]) == [3, 0, 1, 1, 2, 0]
    # no masks in the oldest block: nothing to force
    st, act, stats, _ = update(cfg, [0, 0, 0, 0] + [4] * 4, [(0, 3)] * 8, R=2)
    assert not act.any()
    # a forced EOS counts as EOS
    cfge = cfg4(force_progress=1, eos_id=1)
    st, act, stats, _ = update(cfge, [4, 0, 0, 0], [(1, 2), (0, 6), (0, 6), (0, 6)])
    assert st.tokens[0, 0] == 1 and stats[0, O.ST_EOS] == 1


@pytest.mark.parametrize("s_pe", [0, 2])
def test_forced_progress_bounds_the_steps_on_flat_logits(s_pe):
    """Logits that never clear a threshold: Eq. 1 alone never moves (the
    literal reading), the forced rule retires a block every bl + S_pe steps or
    sooner and the request finishes."""
    bl, n, V = 4, 3, 8
    rng = np.random.default_rng(7)
    for force in (0, 1):
        cfg = cfg4(vocab=V, mask_id=8, eos_id=9, wmax=2, max_blocks=n, s_pe=s_pe, block_len=bl,
                   theta_spawn=0.5, force_progress=force)
        st = one_request_state(cfg, [8] * bl)
        steps = 0
        while st.active[0] == 1 and steps < 100:
            z = rng.standard_normal((cfg.max_slots * bl, V)) * 0.3      # max p ~ 0.2
            O.decode_step(cfg, st, z)
            steps += 1
        if force:
            # each block: bl forced reveals, then at most S_pe post-edit forwards (+1 for the
            # forward that sees it mask-free); nothing else ever happens on these logits
            assert st.active[0] == 2 and steps <= n * (bl + s_pe + 1)
            assert (st.tokens[0] != cfg.mask_id).all()
        else:
            assert steps == 100 and st.L[0] == 0 and (st.tokens[0] == cfg.mask_id).all()
