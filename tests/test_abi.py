"""CPU-only checks of the boundary: the library loads, exports every symbol
the header declares, and rejects bad arguments before touching CUDA."""
import ctypes as C
import os
import re

import pytest

from paper_2607_17652_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

GOOD = dict(max_requests=4, wmax=2, block_len=32, n_q_heads=8, n_kv_heads=2,
            head_dim=128, page_size=64, num_pages=16, max_pages_per_req=4,
            vocab=1024, mask_id=1023, eos_id=1022, max_blocks=8, s_pe=1,
            tau_mask=0.9, tau_edit=0.95, theta_spawn=0.5, sm_scale=0.0)


@pytest.fixture(scope="module", autouse=True)
def built():
    from paper_2607_17652_b200 import build
    build.build()


def test_header_symbols_are_exported():
    hdr = open(os.path.join(ROOT, "include", "flowblock.h")).read()
    declared = set(re.findall(r"\b(fb_[a-z0-9_]+)\s*\(", hdr))
    assert {"fb_pack_wavefronts", "fb_wavefront_attn", "fb_t2t_step",
            "fb_gate_commit"} <= declared
    lib = B.lib()
    for name in declared:
        assert hasattr(lib, name), name
    assert set(B.EXPORTS) >= declared - {"fb_no_such"}
    # every call is bound with explicit argument types (a bare Python int would be cut to 32 bits)
    for name in B.EXPORTS:
        assert getattr(lib, name).argtypes is not None, name


def test_struct_layouts_match_header_order():
    hdr = open(os.path.join(ROOT, "include", "flowblock.h")).read()
    for cls in (B.fb_config, B.fb_tuning, B.fb_state, B.fb_pack, B.fb_host_io, B.fb_device_bufs):
        body = re.search(r"typedef struct \{([^{}]*)\} %s;" % cls.__name__, hdr).group(1)
        body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
        names = re.findall(r"\*?\s*([A-Za-z_][A-Za-z0-9_]*)\s*[;,]", body)
        assert names == [n for n, _ in cls._fields_], cls.__name__


def test_create_validates_configuration():
    ctx = B.Context(**GOOD)
    assert ctx.workspace_bytes() > 0
    bad = [dict(head_dim=96), dict(page_size=32), dict(block_len=24),
           dict(n_kv_heads=3), dict(wmax=0), dict(vocab=1001), dict(wmax=9),
           dict(tau_edit=0.5), dict(s_pe=300), dict(max_requests=-1),
           dict(tau_mask=float("nan")), dict(window_in_pages=2), dict(batch_sync=2),
           dict(delta_literal=2), dict(force_progress=-1), dict(kv_fp8=1), dict(kv_fp8=2),
           dict(kv_fp8=1, window_in_pages=1, head_dim=64)]
    for delta in bad:
        with pytest.raises(B.FlowBlockError):
            B.Context(**dict(GOOD, **delta))
    B.Context(**dict(GOOD, kv_fp8=1, window_in_pages=1))      # 8-bit pages: window in the pages, head_dim 128
    # thresholds the other way round are accepted only with Delta taken literally
    B.Context(**dict(GOOD, tau_edit=0.5, delta_literal=1))
    assert B.lib().fb_create(None, None) == B.FB_ERR_INVALID_ARG
    assert b"null" in B.lib().fb_last_error(None)


def test_window_in_pages_argument_rules():
    lib = B.lib()
    pk = B.fb_pack(*([0x1000] * 9))
    res = B.Context(**dict(GOOD, window_in_pages=1))
    a = [0x1000] * 12
    # page-resident window: window tensors must be null for the attention
    assert lib.fb_wavefront_attn(res.handle, C.byref(pk), 0x1000, 0x1000, 0x1000, 0x1000, 0x1000, 0x1000,
                                 0x1000, 0x1000, 0x1000, None) == B.FB_ERR_INVALID_ARG
    assert b"must be null" in lib.fb_last_error(res.handle)
    assert lib.fb_scatter_window_kv(res.handle, C.byref(pk), 0x1000, None, 0x1000, 0x1000, 0x1000, 0.0,
                                    0x1000, None) == B.FB_ERR_INVALID_ARG
    assert lib.fb_scatter_window_kv(res.handle, C.byref(pk), 0x1000, 0x1008, 0x1000, 0x1000, 0x1000, 0.0,
                                    0x1000, None) == B.FB_ERR_ALIGNMENT
    assert lib.fb_scatter_window_kv(res.handle, C.byref(pk), 0x1000, 0x1000, 0x1000, 0x1000, 0x1000, -1.0,
                                    0x1000, None) == B.FB_ERR_INVALID_ARG
    # slot-order window: window tensors are required
    ctx = B.Context(**GOOD)
    assert lib.fb_wavefront_attn(ctx.handle, C.byref(pk), 0x1000, None, None, 0x1000, 0x1000, 0x1000,
                                 0x1000, 0x1000, 0x1000, None) == B.FB_ERR_INVALID_ARG


def test_null_and_misaligned_arguments_are_rejected_on_the_host():
    ctx = B.Context(**GOOD)
    lib = B.lib()
    st, pk = B.fb_state(), B.fb_pack()
    assert lib.fb_pack_wavefronts(ctx.handle, C.byref(st), C.byref(pk), None, None, None) \
        == B.FB_ERR_INVALID_ARG
    assert b"state.active" in lib.fb_last_error(ctx.handle)
    full_st = B.fb_state(*([0x1000] * 7))
    full_pk = B.fb_pack(*([0x1000] * 9))
    assert lib.fb_pack_wavefronts(ctx.handle, C.byref(full_st), C.byref(full_pk), None,
                                  0x1000, None) == B.FB_ERR_WORKSPACE
    assert lib.fb_pack_wavefronts(ctx.handle, C.byref(full_st), C.byref(full_pk), 0x1010,
                                  0x1000, None) == B.FB_ERR_ALIGNMENT
    args = [0x1000] * 10
    args[0] = 0x1008                                   # q misaligned
    assert lib.fb_wavefront_attn(ctx.handle, C.byref(full_pk), *args) == B.FB_ERR_ALIGNMENT
    assert lib.fb_t2t_step(ctx.handle, C.byref(full_pk), None, C.byref(full_st),
                           *([0x1000] * 6)) == B.FB_ERR_INVALID_ARG
    assert lib.fb_gate_commit(ctx.handle, C.byref(full_pk), None, C.byref(full_st),
                              *([0x1000] * 9)) == B.FB_ERR_INVALID_ARG
    assert lib.fb_step_host(ctx.handle, C.byref(full_st), C.byref(full_pk), None, None,
                            None) == B.FB_ERR_INVALID_ARG
    assert lib.fb_destroy(None) == B.FB_ERR_INVALID_ARG


def test_static_entry_point_rejects_null_members_on_the_host():
    """fb_wavefront_attn_static hands the state and pack arrays to the pack
    kernel: a null member must come back as FB_ERR_INVALID_ARG, not reach a
    launch."""
    ctx = B.Context(**GOOD)
    lib = B.lib()
    for hole in range(7):
        st = B.fb_state(*[None if i == hole else 0x1000 for i in range(7)])
        pk = B.fb_pack(*([0x1000] * 9))
        assert lib.fb_wavefront_attn_static(ctx.handle, C.byref(st), C.byref(pk), *([0x1000] * 7), None) \
            == B.FB_ERR_INVALID_ARG, hole
        assert b"state." in lib.fb_last_error(ctx.handle)
    for hole in range(9):
        st = B.fb_state(*([0x1000] * 7))
        pk = B.fb_pack(*[None if i == hole else 0x1000 for i in range(9)])
        assert lib.fb_wavefront_attn_static(ctx.handle, C.byref(st), C.byref(pk), *([0x1000] * 7), None) \
            == B.FB_ERR_INVALID_ARG, hole
        assert b"pack." in lib.fb_last_error(ctx.handle)
    res = B.Context(**dict(GOOD, window_in_pages=1))
    st, pk = B.fb_state(*([0x1000] * 7)), B.fb_pack(*([0x1000] * 9))
    assert lib.fb_wavefront_attn_static(res.handle, C.byref(st), C.byref(pk), *([0x1000] * 7), None) \
        == B.FB_ERR_UNSUPPORTED


def test_tuning_is_validated_and_resizes_the_workspace():
    ctx = B.Context(**GOOD)
    base = ctx.workspace_bytes()
    ctx.set_tuning(attn_target_items=100000)
    assert ctx.workspace_bytes() >= base
    ctx.set_tuning()                                   # zeros: back to the defaults
    assert ctx.workspace_bytes() == base
    for bad in (dict(attn_target_items=-1), dict(attn_min_chunk_tiles=5000), dict(wait_cycles=-5),
                dict(attn_target_items=(1 << 20) + 1)):
        with pytest.raises(B.FlowBlockError):
            ctx.set_tuning(**bad)
    assert B.lib().fb_set_tuning(ctx.handle, None) == B.FB_ERR_INVALID_ARG


def _llm_cfg(**over):
    return dict(dict(max_requests=16, wmax=3, block_len=64, n_q_heads=32, n_kv_heads=8, head_dim=128,
                     page_size=64, num_pages=16 * 520, max_pages_per_req=520, vocab=1024, mask_id=1023,
                     eos_id=1022, max_blocks=32, s_pe=1, tau_mask=0.9, tau_edit=0.95, theta_spawn=0.5,
                     sm_scale=0.0), **over)


def test_split_pieces_never_exceed_the_workspace_bound():
    """The key-axis split of the attention work list, recomputed on the host by
    the same arithmetic the pack kernel runs: for any batch the units, items
    and split pieces fit what the workspace is sized for.  The hard cases are
    few, long requests (everything becomes split pieces)."""
    import numpy as np
    rg = np.random.default_rng(5)
    # one active long-context request among 16, every 64-aligned prefix in [16384, 32768]
    ctx = B.Context(**_llm_cfg())
    for P in range(16384, 32768 + 1, 64):
        pl = ctx.attn_plan([P], [3])
        for lst in (pl, pl["pair"]):
            assert lst["parts"] <= lst["max_parts"] and lst["items"] <= lst["max_items"], (P, pl)
        assert pl["units"] == 24 and pl["pair"]["units"] == 0 and pl["items"] >= pl["units"]
    # the batch-64 shape with one request of prefix 65536 and four live blocks
    ctx = B.Context(**_llm_cfg(max_requests=64, wmax=4, block_len=32, max_pages_per_req=1030,
                               num_pages=64 * 1030))
    pl = ctx.attn_plan([65536], [4])
    assert pl["pair"]["units"] == 0 and 0 < pl["parts"] <= pl["max_parts"], pl
    ctx.set_tuning(attn_pair=1)                              # quads go to the CTA-pair kernel's list
    pl = ctx.attn_plan([65536], [4])
    assert pl["units"] == 0 and 0 < pl["pair"]["parts"] <= pl["pair"]["max_parts"], pl
    lc = B.Context(tuning=dict(attn_pair=1), **_llm_cfg())
    pl = lc.attn_plan([20000], [3])                          # six Q tiles per KV head: a quad (two records) + a pair
    assert pl["units"] == 8 and pl["pair"]["units"] == 16
    # random batches, several tuning settings
    for target, min_chunk, pair in ((0, 0, 1), (1, 0, 1), (7, 1, 0), (100000, 1, 1), (296, 16, 0), (50, 2, 1)):
        ctx.set_tuning(attn_target_items=target, attn_min_chunk_tiles=min_chunk, attn_pair=pair)
        for _ in range(300):
            n = int(rg.integers(1, 65))
            P = rg.integers(0, 65536, size=n)
            if rg.random() < 0.3:
                P[:] = rg.integers(0, 400)             # many short requests
            w = rg.integers(0, 5, size=n)
            pl = ctx.attn_plan(P, w)
            for lst in (pl, pl["pair"]):
                assert lst["units"] <= lst["max_units"], pl
                assert lst["items"] <= lst["max_items"], pl
                assert lst["parts"] <= lst["max_parts"], (target, min_chunk, pl)
            assert (pl["pair"]["units"] == 0) == (pair == 0 or (np.asarray(w) < 4).all())
    assert B.lib().fb_attn_plan_host(ctx.handle, None, None, 0, None) == B.FB_ERR_INVALID_ARG
