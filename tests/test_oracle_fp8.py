"""Pins of the oracle's 8-bit (FP8 E4M3) KV pages: the code table and the
rounding against the format's definition and against a library conversion,
hand-worked ties / subnormals / saturation, and the two functions built on
them against the bf16-path functions they must reduce to (CPU)."""
import numpy as np
import torch

from oracle import flowblock_oracle as O
from paper_2607_17652_b200 import synth
from tests import harness as H


def test_decode_table_is_the_e4m3_format():
    codes = np.arange(256, dtype=np.uint8)
    v = O.e4m3_decode(codes)
    # hand-checked entries of the format: zero, smallest subnormal, largest subnormal,
    # smallest normal, one, largest finite, NaN; sign bit mirrors
    assert v[0x00] == 0.0 and v[0x01] == 2.0 ** -9 and v[0x07] == 7 * 2.0 ** -9
    assert v[0x08] == 2.0 ** -6 and v[0x38] == 1.0 and v[0x39] == 1.125 and v[0x40] == 2.0
    assert v[0x7E] == 448.0 and np.isnan(v[0x7F]) and np.isnan(v[0xFF])
    np.testing.assert_array_equal(v[0x80:0xFF], -v[0x00:0x7F])
    assert (np.diff(v[:0x7F]) > 0).all()                      # the positive codes are ordered
    # the library's float8 type reads the same 256 values
    lib = torch.from_numpy(codes).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    np.testing.assert_array_equal(np.nan_to_num(v, nan=1e9), np.nan_to_num(lib, nan=1e9))


def test_rounding_round_trips_and_hand_worked_cases():
    codes = np.array([c for c in range(256) if c & 0x7F != 0x7F], np.uint8)
    np.testing.assert_array_equal(O.e4m3_round(O.e4m3_decode(codes)), codes)     # representable values are fixed points
    dec = lambda y: O.e4m3_decode(O.e4m3_round(np.array(y, np.float64))).tolist()
    # ties go to the even mantissa: 1.0625 is half way 1.0 (m=0) / 1.125 (m=1); 1.1875 half way 1.125 / 1.25 (m=2)
    assert dec([1.0625, 1.1875, -1.0625]) == [1.0, 1.25, -1.0]
    assert dec([1.07, 1.18]) == [1.125, 1.125]
    # subnormals: grid 2^-9; 2^-10 is a tie with zero (even), just above it rounds up
    assert dec([2.0 ** -10, 2.0 ** -10 * 1.01, 1.5 * 2.0 ** -9, 2.5 * 2.0 ** -9]) == \
        [0.0, 2.0 ** -9, 2 * 2.0 ** -9, 2 * 2.0 ** -9]
    # carry into the next binade and into the normal range
    assert dec([1.97, 7.9 * 2.0 ** -9]) == [2.0, 2.0 ** -6]
    # saturation, both signs; the largest value that still rounds to 448 without it
    assert dec([1000.0, -1e9, 464.0, 449.0, 431.9]) == [448.0, -448.0, 448.0, 448.0, 416.0]
    # half a grid step is the largest error inside the range
    rg = np.random.default_rng(3)
    y = rg.uniform(-448, 448, size=20000)
    err = np.abs(O.e4m3_decode(O.e4m3_round(y)) - y)
    step = np.exp2(np.floor(np.log2(np.maximum(np.abs(y), 2.0 ** -6))) - 3)
    assert (err <= step / 2).all()
    assert (np.diff(O.e4m3_decode(O.e4m3_round(np.sort(y)))) >= 0).all()          # monotone


def test_rounding_agrees_with_the_library_conversion():
    rg = np.random.default_rng(11)
    y = (rg.normal(size=300000) * np.exp2(rg.integers(-12, 9, size=300000))).astype(np.float32)
    y = y[np.abs(y) <= 448.0]
    lib = torch.from_numpy(y).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    np.testing.assert_array_equal(O.e4m3_round(y.astype(np.float64)), lib)


def test_quantize_divides_in_binary32_and_is_scale_invariant():
    rg = np.random.default_rng(5)
    x = rg.normal(size=5000)
    s = np.float32(0.0137)
    np.testing.assert_array_equal(O.e4m3_quantize(x, s), O.e4m3_quantize(x * 8.0, s * np.float32(8.0)))
    np.testing.assert_array_equal(O.e4m3_quantize(x, np.float32(1.0)), O.e4m3_round(x.astype(np.float32)))
    # the stored value read back is within half a code step of x (or saturated)
    back = O.e4m3_decode(O.e4m3_quantize(x, s)) * float(s)
    step = np.exp2(np.floor(np.log2(np.maximum(np.abs(x / float(s)), 2.0 ** -6))) - 3) * float(s)
    inside = np.abs(x / float(s)) <= 448
    assert (np.abs(back - x)[inside] <= step[inside] / 2 * (1 + 1e-6)).all()
    assert (np.abs(back[~inside]) == 448 * float(s)).all()
    # a quotient that binary32 rounds onto a tie: x = 17, scale = 16 -> 1.0625 exactly -> even mantissa
    assert O.e4m3_decode(O.e4m3_quantize(np.array([17.0]), np.float32(16.0)))[0] == 1.0


def _case(seed=5):
    wl = synth.tiny_workload(n_requests=4, wmax=3, w_lo=1, w_hi=3, prefix_lo=3, prefix_hi=150,
                             n_q_heads=4, n_kv_heads=2, head_dim=8, max_blocks=8, block_len=4)
    stc = synth.make_structure(wl, seed)
    tokens = synth.make_tokens(stc)
    cfg = H.oracle_cfg(stc)
    st = H.oracle_state(stc, tokens)
    pk = O.pack_wavefronts(cfg, st)
    q, kw, vw, kp, vp = (H.f64(t) for t in synth.make_attn_inputs(stc))
    return wl, stc, cfg, st, pk, q, kw, vw, kp, vp


def test_fp8_functions_reduce_to_the_bf16_path_on_representable_values():
    """With scale 1 and K/V that E4M3 represents exactly, nothing is lost: the
    8-bit scatter stores exactly those values and the 8-bit attention equals
    the plain attention over the page-resident window."""
    wl, stc, cfg, st, pk, q, kw, vw, kp, vp = _case()
    snap = lambda a: O.e4m3_decode(O.e4m3_round(a))            # any value -> a representable one
    kw, vw, kp, vp = snap(kw), snap(vw), snap(kp), snap(vp)
    one = np.ones(wl.n_kv_heads, np.float32)
    kp8, vp8 = O.e4m3_round(kp), O.e4m3_round(vp)
    O.scatter_window_kv_fp8(cfg, pk, kw, vw, kp8, vp8, one, one, st.page_table)
    O.scatter_window_kv(cfg, pk, kw, vw, kp, vp, st.page_table)
    np.testing.assert_array_equal(O.e4m3_decode(kp8), kp)
    np.testing.assert_array_equal(O.e4m3_decode(vp8), vp)
    ref = O.wavefront_attn(cfg, pk, q, None, None, kp, vp, st.page_table)
    got = O.wavefront_attn_fp8(cfg, pk, q, kp8, vp8, one, one, st.page_table)
    np.testing.assert_array_equal(got, ref)


def test_fp8_scales_act_on_scores_and_outputs():
    """value = code * scale: doubling a head's V scale doubles that head's
    outputs and nothing else; a K scale is the same as scaling the queries of
    that head's group; placement and untouched positions as in the bf16 path."""
    wl, stc, cfg, st, pk, q, kw, vw, kp, vp = _case(seed=9)
    rg = np.random.default_rng(2)
    ks = rg.uniform(0.01, 0.05, size=wl.n_kv_heads).astype(np.float32)
    vs = rg.uniform(0.01, 0.05, size=wl.n_kv_heads).astype(np.float32)
    kp8, vp8 = O.e4m3_quantize(kp, ks[None, :, None, None]), O.e4m3_quantize(vp, vs[None, :, None, None])
    before_k = kp8.copy()
    O.scatter_window_kv_fp8(cfg, pk, kw, vw, kp8, vp8, ks, vs, st.page_table)
    # exactly the live window positions changed (same set as the bf16 scatter touches)
    kpb, vpb = kp.copy(), vp.copy()
    O.scatter_window_kv(cfg, pk, kw + 1000.0, vw, kpb, vpb, st.page_table)
    touched = (kpb != kp).any(axis=(1, 3))                    # [page, offset]
    same = (kp8 == before_k).all(axis=(1, 3))
    assert (same | touched).all() and touched.sum() == pk.n_live * wl.block_len
    base = O.wavefront_attn_fp8(cfg, pk, q, kp8, vp8, ks, vs, st.page_table)
    G = wl.n_q_heads // wl.n_kv_heads
    vs2 = vs.copy(); vs2[1] *= 2
    got = O.wavefront_attn_fp8(cfg, pk, q, kp8, vp8, ks, vs2, st.page_table)
    np.testing.assert_allclose(got[:, G:], 2 * base[:, G:], rtol=1e-13)
    np.testing.assert_array_equal(got[:, :G], base[:, :G])
    ks2 = ks.copy(); ks2[0] *= 4
    q2 = q.copy(); q2[:, :G] *= 4
    np.testing.assert_allclose(O.wavefront_attn_fp8(cfg, pk, q, kp8, vp8, ks2, vs, st.page_table),
                               O.wavefront_attn_fp8(cfg, pk, q2, kp8, vp8, ks, vs, st.page_table), rtol=1e-12)
    # against the unquantised attention: the error is what half a code step on K and V allows
    O.scatter_window_kv(cfg, pk, kw, vw, kp, vp, st.page_table)
    exact = O.wavefront_attn(cfg, pk, q, None, None, kp, vp, st.page_table)
    live = pk.n_live * wl.block_len
    rel = np.linalg.norm(base[:live] - exact[:live]) / np.linalg.norm(exact[:live])
    assert 1e-4 < rel < 0.08


def test_synthetic_fp8_pools_are_plain_bytes_with_finite_values():
    wl = synth.tiny_workload()
    stc = synth.make_structure(wl)
    k8, v8, ks, vs = synth.make_fp8_kv(stc)
    assert k8.dtype == torch.uint8 and k8.shape == (stc.num_pages, wl.n_kv_heads, 64, wl.head_dim)
    assert np.isfinite(O.e4m3_decode(k8.numpy())).all() and np.isfinite(O.e4m3_decode(v8.numpy())).all()
    assert ks.dtype == torch.float32 and len(ks) == wl.n_kv_heads and (vs > 0).all()
    assert len(np.unique(k8.numpy())) > 100                    # the codes in use span the format


def test_weight_norms_closed_forms():
    """sum w^2 is 1/n for the n equal weights of a zero query and 1 when one key dominates."""
    wl, stc, cfg, st, pk, q, kw, vw, kp, vp = _case(seed=4)
    O.scatter_window_kv(cfg, pk, kw, vw, kp, vp, st.page_table)
    n2 = O.wavefront_attn_weight_norms(cfg, pk, np.zeros_like(q), None, kp, st.page_table)
    b = wl.block_len
    for slot in range(pk.n_live):
        np.testing.assert_allclose(n2[slot * b:(slot + 1) * b], 1.0 / int(pk.slot_kv_len[slot]), rtol=1e-12)
    assert not n2[pk.n_live * b:].any()
    kp2 = kp.copy()
    r = int(pk.slot_req[0])
    kp2[int(st.page_table[r, 0]), :, 0, :] = 50.0                 # position 0 of request r
    n2 = O.wavefront_attn_weight_norms(cfg, pk, np.ones_like(q), None, kp2, st.page_table)
    assert int(st.prefix_len[r]) > 0 and np.abs(n2[:b] - 1.0).max() < 1e-9
