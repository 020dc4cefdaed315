"""CPU pins for the oracle's packing and attention (no GPU, no CUDA path).

Each test checks the oracle against something other than itself: brute-force
enumeration, the literal dense mask of Eq. 5 in the paper's own cache layout,
closed forms, and the structural invariants of Sec. 3.1 / 3.2.
"""
import os

import numpy as np
import pytest

from oracle import flowblock_oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def small_cfg(R=3, W=3, b=4, Hq=2, Hkv=1, d=8, ps=4, n=6):
    return O.Config(max_requests=R, wmax=W, block_len=b, n_q_heads=Hq,
                    n_kv_heads=Hkv, head_dim=d, page_size=ps, vocab=16,
                    mask_id=15, eos_id=14, max_blocks=n)


def random_state(cfg, rng, prefixes=None, wlive=None, active=None):
    R, W, b, n = cfg.max_requests, cfg.wmax, cfg.block_len, cfg.max_blocks
    P = np.array(prefixes if prefixes is not None
                 else rng.integers(0, 20, size=R), np.int32)
    Wr = np.array(wlive if wlive is not None
                  else rng.integers(0, W + 1, size=R), np.int32)
    L = rng.integers(0, n - W + 1, size=R).astype(np.int32)
    act = np.array(active if active is not None
                   else rng.integers(0, 3, size=R), np.int32)
    need = (P + W * b + cfg.page_size - 1) // cfg.page_size
    cfg.max_pages_per_req = int(need.max())
    cfg.num_pages = int(need.sum()) + 3
    perm = rng.permutation(cfg.num_pages).astype(np.int32)
    pt = np.zeros((R, cfg.max_pages_per_req), np.int32)
    off = 0
    for r in range(R):
        pt[r, :need[r]] = perm[off:off + need[r]]
        off += need[r]
    tokens = rng.integers(0, cfg.vocab, size=(R, n * b)).astype(np.int32)
    return O.State(act, P, L, (L + Wr).astype(np.int32), tokens,
                   np.zeros((R, W), np.uint8), pt)


def random_kv(cfg, rng):
    S, b = cfg.max_slots, cfg.block_len
    q = rng.standard_normal((S * b, cfg.n_q_heads, cfg.head_dim))
    kw = rng.standard_normal((S * b, cfg.n_kv_heads, cfg.head_dim))
    vw = rng.standard_normal((S * b, cfg.n_kv_heads, cfg.head_dim))
    kp = rng.standard_normal((cfg.num_pages, cfg.n_kv_heads, cfg.page_size,
                              cfg.head_dim))
    vp = rng.standard_normal(kp.shape)
    return q, kw, vw, kp, vp


# ------------------------------------------------------------------ pack
def test_window_capacity_worked_value():
    for line in open(os.path.join(GOLD, "window_capacity.txt")):
        if line.startswith("#") or not line.strip():
            continue
        W, bl, q = map(int, line.split())
        assert O.Config(max_requests=1, wmax=W, block_len=bl).q_capacity == q


def test_pack_bruteforce_enumeration():
    rng = np.random.default_rng(1)
    for trial in range(50):
        cfg = small_cfg(R=int(rng.integers(1, 6)), W=int(rng.integers(1, 5)),
                        b=int(rng.integers(1, 5)), n=8)
        st = random_state(cfg, rng)
        pk = O.pack_wavefronts(cfg, st)
        b = cfg.block_len
        # brute force: the set of live (request, block) pairs, in order
        want = [(r, g) for r in range(cfg.max_requests) if st.active[r] == 1
                for g in range(st.L[r], st.R[r])]
        assert pk.n_live == len(want) <= cfg.max_slots
        got = [(int(pk.slot_req[i]), int(st.L[pk.slot_req[i]] + pk.slot_s[i]))
               for i in range(pk.n_live)]
        assert got == want
        assert (pk.slot_req[pk.n_live:] == -1).all()
        assert (pk.qtok[pk.n_live * b:] == cfg.mask_id).all()
        assert (pk.pos[pk.n_live * b:] == 0).all()
        for i, (r, g) in enumerate(want):
            # Eq. 4: qtok = x[r, o_r + ...], pos = o_r + ... (absolute ids)
            assert (pk.qtok[i * b:(i + 1) * b] ==
                    st.tokens[r, g * b:(g + 1) * b]).all()
            s = g - st.L[r]
            assert (pk.pos[i * b:(i + 1) * b] ==
                    st.prefix_len[r] + s * b + np.arange(b)).all()
            assert pk.slot_kv_len[i] == st.prefix_len[r] + (s + 1) * b
            assert bool(pk.slot_flags[i] & O.FLAG_OLDEST) == (g == st.L[r])
            assert bool(pk.slot_flags[i] & O.FLAG_FRONTIER) == (g == st.R[r] - 1)
            assert pk.req_slot_begin[r] <= i < pk.req_slot_begin[r + 1]
        # positions strictly increase inside a request
        for r in range(cfg.max_requests):
            lo, hi = pk.req_slot_begin[r] * b, pk.req_slot_begin[r + 1] * b
            assert (np.diff(pk.pos[lo:hi]) == 1).all()


# ------------------------------------------------------------- attention
def to_physical(cfg, st, pk, q, kw, vw, kp, vp, C, rng):
    """The paper's layout: per request a cache of C rows, prefix at [0,o_b),
    garbage in the stale middle, the whole q = W*bl window at the tail."""
    R, W, b = cfg.max_requests, cfg.wmax, cfg.block_len
    qcap = W * b
    t = C - qcap
    q_req = rng.standard_normal((R, qcap, cfg.n_q_heads, cfg.head_dim))
    k_phys = 50.0 * rng.standard_normal((R, C, cfg.n_kv_heads, cfg.head_dim))
    v_phys = 50.0 * rng.standard_normal((R, C, cfg.n_kv_heads, cfg.head_dim))
    for r in range(R):
        for j in range(st.prefix_len[r]):
            pg = st.page_table[r, j // cfg.page_size]
            k_phys[r, j] = kp[pg, :, j % cfg.page_size]
            v_phys[r, j] = vp[pg, :, j % cfg.page_size]
        for i in range(pk.req_slot_begin[r], pk.req_slot_begin[r + 1]):
            s = pk.slot_s[i]
            q_req[r, s * b:(s + 1) * b] = q[i * b:(i + 1) * b]
            k_phys[r, t + s * b:t + (s + 1) * b] = kw[i * b:(i + 1) * b]
            v_phys[r, t + s * b:t + (s + 1) * b] = vw[i * b:(i + 1) * b]
    return q_req, k_phys, v_phys


@pytest.mark.parametrize("prefixes,wlive", [([5, 9, 0], [3, 2, 1]),
                                            ([13, 4, 7], [1, 3, 3]),
                                            ([1, 2, 16], [2, 0, 3])])
def test_attention_equals_literal_eq5_dense_mask(prefixes, wlive):
    rng = np.random.default_rng(7)
    cfg = small_cfg()
    st = random_state(cfg, rng, prefixes, wlive, active=[1, 1, 1])
    pk = O.pack_wavefronts(cfg, st)
    q, kw, vw, kp, vp = random_kv(cfg, rng)
    out = O.wavefront_attn(cfg, pk, q, kw, vw, kp, vp, st.page_table)
    C = max(prefixes) + cfg.q_capacity + 3          # a stale middle exists
    q_req, k_phys, v_phys = to_physical(cfg, st, pk, q, kw, vw, kp, vp, C, rng)
    ref = O.dense_mask_attn_bruteforce(cfg, st.prefix_len, wlive, q_req,
                                       k_phys, v_phys, C)
    b = cfg.block_len
    for i in range(pk.n_live):
        r, s = pk.slot_req[i], pk.slot_s[i]
        np.testing.assert_allclose(out[i * b:(i + 1) * b],
                                   ref[r, s * b:(s + 1) * b],
                                   rtol=0, atol=1e-12)


def test_attention_closed_forms():
    rng = np.random.default_rng(3)
    cfg = small_cfg(Hq=4, Hkv=2)
    st = random_state(cfg, rng, [5, 9, 2], [3, 2, 3], active=[1, 1, 1])
    pk = O.pack_wavefronts(cfg, st)
    q, kw, vw, kp, vp = random_kv(cfg, rng)
    b, G = cfg.block_len, cfg.n_q_heads // cfg.n_kv_heads
    # (1) zero queries: all scores tie, output = mean over exactly the
    #     P_r + (s+1) bl visible V rows
    out = O.wavefront_attn(cfg, pk, np.zeros_like(q), kw, vw, kp, vp,
                           st.page_table)
    for i in range(pk.n_live):
        r, s = pk.slot_req[i], pk.slot_s[i]
        rows = [vp[st.page_table[r, j // cfg.page_size], :, j % cfg.page_size]
                for j in range(st.prefix_len[r])]
        first = pk.req_slot_begin[r]
        rows += [vw[(first + s2) * b + t] for s2 in range(s + 1)
                 for t in range(b)]
        assert len(rows) == st.prefix_len[r] + (s + 1) * b == pk.slot_kv_len[i]
        mean = np.mean(rows, axis=0)                  # [Hkv, d]
        for h in range(cfg.n_q_heads):
            np.testing.assert_allclose(out[i * b:(i + 1) * b, h],
                                       np.tile(mean[h // G], (b, 1)),
                                       atol=1e-12)
    # (2) constant V: output is that constant whatever the scores
    out = O.wavefront_attn(cfg, pk, q, kw, np.full_like(vw, 2.5), kp,
                           np.full_like(vp, 2.5), st.page_table)
    np.testing.assert_allclose(out[:pk.n_live * b], 2.5, atol=1e-12)
    # (3) one key aligned with the query at score +40: output ~ its V row
    i = 1                                            # request 0, slot 1
    row = 1 * b + 2                                  # window key in block 1
    q2 = np.zeros_like(q)
    kw2 = np.zeros_like(kw)
    q2[0:2 * b, :, 0] = 40.0 * np.sqrt(cfg.head_dim)  # slots 0 and 1
    kw2[row, :, 0] = 1.0
    out = O.wavefront_attn(cfg, pk, q2, kw2, vw, np.zeros_like(kp), vp,
                           st.page_table)
    for h in range(cfg.n_q_heads):
        np.testing.assert_allclose(out[i * b:(i + 1) * b, h],
                                   np.tile(vw[row, h // G], (b, 1)), atol=1e-9)
    # ... while the block to its left cannot see that key: all of its scores
    # are zero, so it still returns the mean of its own visible V rows
    rows = [vp[st.page_table[0, j // cfg.page_size], :, j % cfg.page_size]
            for j in range(st.prefix_len[0])] + [vw[t] for t in range(b)]
    mean = np.mean(rows, axis=0)
    for h in range(cfg.n_q_heads):
        np.testing.assert_allclose(out[0:b, h], np.tile(mean[h // G], (b, 1)),
                                   atol=1e-12)


def test_attention_isolation_and_block_causality():
    rng = np.random.default_rng(11)
    cfg = small_cfg()
    st = random_state(cfg, rng, [6, 3, 10], [3, 2, 1], active=[1, 1, 1])
    pk = O.pack_wavefronts(cfg, st)
    q, kw, vw, kp, vp = random_kv(cfg, rng)
    b = cfg.block_len
    base = O.wavefront_attn(cfg, pk, q, kw, vw, kp, vp, st.page_table)
    # perturb everything that belongs to requests 1 and 2 or to padding
    kw2, vw2, kp2, vp2 = kw.copy(), vw.copy(), kp.copy(), vp.copy()
    lo = pk.req_slot_begin[1] * b
    kw2[lo:] += 100.0
    vw2[lo:] -= 100.0
    own = set(st.page_table[0, :(6 + cfg.page_size - 1) // cfg.page_size])
    for pg in range(cfg.num_pages):
        if pg not in own:
            kp2[pg] += 9.0
            vp2[pg] -= 9.0
    # ... and the part of request 0's last prefix page beyond its prefix
    last = st.page_table[0, 6 // cfg.page_size]
    kp2[last, :, 6 % cfg.page_size:] = 77.0
    vp2[last, :, 6 % cfg.page_size:] = -77.0
    out = O.wavefront_attn(cfg, pk, q, kw2, vw2, kp2, vp2, st.page_table)
    assert np.array_equal(out[:3 * b], base[:3 * b])     # bit for bit
    # block causality: altering blocks to the right never changes a block
    kw3, vw3 = kw.copy(), vw.copy()
    kw3[2 * b:3 * b] += 5.0
    vw3[2 * b:3 * b] += 5.0
    out = O.wavefront_attn(cfg, pk, q, kw3, vw3, kp, vp, st.page_table)
    assert np.array_equal(out[:2 * b], base[:2 * b])
    assert not np.array_equal(out[2 * b:3 * b], base[2 * b:3 * b])
    # leftmost block of a 3-block window == the same block decoded serially
    # (window of one block): exact frozen-prefix reuse (Sec. 3.1)
    st1 = st.copy()
    st1.R[:] = st1.L + np.array([1, 1, 1])
    pk1 = O.pack_wavefronts(cfg, st1)
    q1 = np.zeros_like(q); k1 = np.zeros_like(kw); v1 = np.zeros_like(vw)
    for i1 in range(pk1.n_live):
        i0 = pk.req_slot_begin[pk1.slot_req[i1]]
        q1[i1 * b:(i1 + 1) * b] = q[i0 * b:(i0 + 1) * b]
        k1[i1 * b:(i1 + 1) * b] = kw[i0 * b:(i0 + 1) * b]
        v1[i1 * b:(i1 + 1) * b] = vw[i0 * b:(i0 + 1) * b]
    ser = O.wavefront_attn(cfg, pk1, q1, k1, v1, kp, vp, st.page_table)
    for i1 in range(pk1.n_live):
        i0 = pk.req_slot_begin[pk1.slot_req[i1]]
        np.testing.assert_allclose(ser[i1 * b:(i1 + 1) * b],
                                   base[i0 * b:(i0 + 1) * b], atol=1e-13)


def test_attention_matches_library_sdpa_when_unmasked():
    """Special case that reduces to a library routine: one request, one live
    block, no prefix -> plain bidirectional attention over the block."""
    import torch
    rng = np.random.default_rng(5)
    cfg = small_cfg(R=1, W=1, b=4, Hq=2, Hkv=2, d=8)
    st = random_state(cfg, rng, [0], [1], active=[1])
    pk = O.pack_wavefronts(cfg, st)
    q, kw, vw, kp, vp = random_kv(cfg, rng)
    out = O.wavefront_attn(cfg, pk, q, kw, vw, kp, vp, st.page_table)
    tq = torch.from_numpy(q).permute(1, 0, 2)[None]      # [1, H, b, d]
    tk = torch.from_numpy(kw).permute(1, 0, 2)[None]
    tv = torch.from_numpy(vw).permute(1, 0, 2)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv)
    np.testing.assert_allclose(out, ref[0].permute(1, 0, 2).numpy(),
                               atol=1e-12)


def test_bf16_widening_is_exact():
    import torch
    x = torch.randn(1000, dtype=torch.float32).to(torch.bfloat16)
    bits = x.view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(O.bf16_bits_to_f64(bits),
                                  x.to(torch.float64).numpy())
