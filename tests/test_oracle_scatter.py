"""Pins of the oracle's Eq. 6 data movement (window K/V resident in the pages)
and of its rotary embedding, against brute force and textbook cases (CPU)."""
import numpy as np

from oracle import flowblock_oracle as O
from paper_2607_17652_b200 import synth
from tests import harness as H


def _case(seed=5, **kw):
    wl = synth.tiny_workload(n_requests=4, wmax=3, w_lo=1, w_hi=3, prefix_lo=3, prefix_hi=150,
                             n_q_heads=4, n_kv_heads=2, head_dim=8, max_blocks=8, block_len=4, **kw)
    stc = synth.make_structure(wl, seed)
    tokens = synth.make_tokens(stc)
    cfg = H.oracle_cfg(stc)
    st = H.oracle_state(stc, tokens)
    pk = O.pack_wavefronts(cfg, st)
    q, kw_, vw, kp, vp = (H.f64(t) for t in synth.make_attn_inputs(stc))
    return wl, stc, cfg, st, pk, q, kw_, vw, kp, vp


def test_scatter_places_every_live_window_position_and_nothing_else():
    wl, stc, cfg, st, pk, q, kw, vw, kp, vp = _case()
    kp0, vp0 = kp.copy(), vp.copy()
    O.scatter_window_kv(cfg, pk, kw, vw, kp, vp, st.page_table)
    touched = np.zeros(kp.shape[:1] + kp.shape[2:3], bool)          # [page, offset]
    b, ps = wl.block_len, wl.page_size
    n = 0
    for r in range(wl.n_requests):
        if st.active[r] != 1:
            continue
        for g in range(int(st.L[r]), int(st.R[r])):
            slot = n
            n += 1
            for t in range(b):
                pos = int(st.prefix_len[r]) + (g - int(st.L[r])) * b + t     # o_r + s*bl + t
                page, off = int(st.page_table[r, pos // ps]), pos % ps
                np.testing.assert_array_equal(kp[page, :, off], kw[slot * b + t])
                np.testing.assert_array_equal(vp[page, :, off], vw[slot * b + t])
                assert not touched[page, off]
                touched[page, off] = True
    assert n == pk.n_live and touched.sum() == n * b
    keep = ~touched
    np.testing.assert_array_equal(kp.transpose(0, 2, 1, 3)[keep], kp0.transpose(0, 2, 1, 3)[keep])
    np.testing.assert_array_equal(vp.transpose(0, 2, 1, 3)[keep], vp0.transpose(0, 2, 1, 3)[keep])


def test_attention_over_resident_window_equals_slot_order_window():
    wl, stc, cfg, st, pk, q, kw, vw, kp, vp = _case(seed=9)
    ref = O.wavefront_attn(cfg, pk, q, kw, vw, kp, vp, st.page_table)
    O.scatter_window_kv(cfg, pk, kw, vw, kp, vp, st.page_table)
    got = O.wavefront_attn(cfg, pk, q, None, None, kp, vp, st.page_table)
    np.testing.assert_array_equal(got, ref)


def test_pointer_bump_commit_equals_copy_at_commit():
    """Retiring blocks after a scatter needs no copy: the pools equal those of
    the copy-at-commit path on every frozen position."""
    wl, stc, cfg, st, pk, q, kw, vw, kp, vp = _case(seed=3)
    stats = np.zeros((cfg.max_slots, 6), np.int32)          # no masks, no updates: every block finished
    st_a = H.oracle_state(stc, st.tokens)
    st_b = H.oracle_state(stc, st.tokens)
    st_a.tokens[st_a.tokens == cfg.mask_id] = 1
    st_b.tokens[:] = st_a.tokens
    kpa, vpa, kpb, vpb = kp.copy(), vp.copy(), kp.copy(), vp.copy()
    na, _, _ = O.gate_commit(cfg, pk, stats, st_a, kw, vw, kpa, vpa)
    O.scatter_window_kv(cfg, pk, kw, vw, kpb, vpb, st_b.page_table)
    nb, _, _ = O.gate_commit(cfg, pk, stats, st_b)            # pointer bump only
    np.testing.assert_array_equal(na, nb)
    assert na.sum() > 0
    ps = wl.page_size
    for r in range(wl.n_requests):
        for pos in range(int(st_a.prefix_len[r])):
            page, off = int(st_a.page_table[r, pos // ps]), pos % ps
            np.testing.assert_array_equal(kpa[page, :, off], kpb[page, :, off])
            np.testing.assert_array_equal(vpa[page, :, off], vpb[page, :, off])


def test_rope_textbook_cases():
    rg = np.random.default_rng(1)
    x = rg.normal(size=(3, 16))
    np.testing.assert_allclose(O.rope_rotate(x, 0, 10000.0), x, atol=0)
    # d = 2: a plain rotation by `pos` radians
    np.testing.assert_allclose(O.rope_rotate(np.array([1.0, 0.0]), 0.5, 10000.0),
                               [np.cos(0.5), np.sin(0.5)], atol=1e-15)
    # first pair turns by pos, the last by pos * base^(-(d-2)/d)
    e0 = np.zeros(8); e0[0] = 1.0
    y = O.rope_rotate(e0, 3, 100.0)
    np.testing.assert_allclose([y[0], y[4]], [np.cos(3.0), np.sin(3.0)], atol=1e-15)
    e3 = np.zeros(8); e3[3] = 1.0
    y = O.rope_rotate(e3, 3, 100.0)
    np.testing.assert_allclose([y[3], y[7]], [np.cos(3 * 100.0 ** -0.75), np.sin(3 * 100.0 ** -0.75)], atol=1e-15)
    # norms are kept, and q.k depends on the offset between the positions only
    np.testing.assert_allclose(np.linalg.norm(O.rope_rotate(x, 777, 10000.0), axis=-1),
                               np.linalg.norm(x, axis=-1), rtol=1e-13)
    q, k = rg.normal(size=16), rg.normal(size=16)
    a = O.rope_rotate(q, 40, 10000.0) @ O.rope_rotate(k, 33, 10000.0)
    b = O.rope_rotate(q, 1040, 10000.0) @ O.rope_rotate(k, 1033, 10000.0)
    np.testing.assert_allclose(a, b, rtol=1e-10)


def test_scatter_with_rope_rotates_keys_only():
    wl, stc, cfg, st, pk, q, kw, vw, kp, vp = _case(seed=11)
    O.scatter_window_kv(cfg, pk, kw, vw, kp, vp, st.page_table, rope_base=10000.0)
    b, ps = wl.block_len, wl.page_size
    for slot in range(pk.n_live):
        r = int(pk.slot_req[slot])
        for t in range(b):
            pos = int(pk.slot_pos0[slot]) + t
            page, off = int(st.page_table[r, pos // ps]), pos % ps
            np.testing.assert_allclose(kp[page, :, off], O.rope_rotate(kw[slot * b + t], pos, 10000.0), atol=0)
            np.testing.assert_array_equal(vp[page, :, off], vw[slot * b + t])


def test_embed_gather_brute_force():
    wl, stc, cfg, st, pk, q, kw, vw, kp, vp = _case(seed=21)
    rg = np.random.default_rng(3)
    table = rg.normal(size=(wl.vocab, 12))
    x = O.embed_gather(cfg, pk, table)
    b = wl.block_len
    slot = 0
    for r in range(wl.n_requests):
        if st.active[r] != 1:
            continue
        for g in range(int(st.L[r]), int(st.R[r])):
            for t in range(b):
                np.testing.assert_array_equal(x[slot * b + t], table[st.tokens[r, g * b + t]])
            slot += 1
    assert slot == pk.n_live and not x[slot * b:].any()


def test_lm_head_rows_closed_forms():
    wl, stc, cfg, st, pk, q, kw, vw, kp, vp = _case(seed=4)
    n = pk.n_live * wl.block_len
    rows, V, hid = cfg.max_slots * wl.block_len, wl.vocab, 16
    rg = np.random.default_rng(8)
    # hidden state = unit vector e_0, so the logits of a row are column 0 of the weights:
    # one entry a, the others 0  ->  p = e^a / (e^a + V - 1)
    for a in (0.0, 2.0, 5.0):
        w = np.zeros((V, hid)); w[:, 1:] = rg.normal(size=(V, hid - 1))
        w[7, 0] = a
        x = np.zeros((rows, hid)); x[:, 0] = 1.0
        xhat, conf = O.lm_head_rows(cfg, pk, x, w)
        want = np.exp(a) / (np.exp(a) + V - 1)
        np.testing.assert_allclose(conf[:n], want, rtol=1e-12)
        assert (xhat[:n] == (7 if a > 0 else 0)).all()          # a = 0: V-way tie -> index 0
        assert (xhat[n:] == -1).all() and not conf[n:].any()
    # generic inputs: a permutation of the vocabulary permutes the winners, keeps the confidences
    w = rg.normal(size=(V, hid)) / 4.0
    x = rg.normal(size=(rows, hid))
    xhat, conf = O.lm_head_rows(cfg, pk, x, w)
    perm = rg.permutation(V)
    xhat2, conf2 = O.lm_head_rows(cfg, pk, x, w[perm])
    np.testing.assert_array_equal(perm[xhat2[:n]], xhat[:n])
    np.testing.assert_allclose(conf2[:n], conf[:n], rtol=1e-12)
    # confidence of the winner against a direct evaluation of one row
    z = w @ x[3]
    np.testing.assert_allclose(conf[3], 1.0 / np.exp(z - z.max()).sum(), rtol=1e-12)
    assert xhat[3] == int(np.argmax(z))
