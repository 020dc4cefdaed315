"""Guard bands around every buffer the library writes (the sanitizer is not
available on the test machines, so this stands in for its out-of-bounds check):
each output, the pack arrays, the workspace and the KV pools sit inside a larger
allocation whose margins hold a byte pattern; after whole decode steps -- bf16
pages, the window in the pages, 8-bit pages, the CTA-pair kernel, forced key-axis
splits -- every margin must still hold it."""
import numpy as np
import pytest
import torch

from paper_2607_17652_b200 import binding as B
from paper_2607_17652_b200 import synth
from tests import harness as H

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
GUARD = 4096
PATTERN = 0xA5


class Guarded:
    """Device tensors carved out of guarded allocations."""

    def __init__(self):
        self.raw = []

    def like(self, t: torch.Tensor) -> torch.Tensor:
        """A device copy of `t` with GUARD bytes of pattern on either side (256-byte aligned start)."""
        n = t.numel() * t.element_size()
        n_pad = (n + 255) // 256 * 256
        raw = torch.full((GUARD + n_pad + GUARD,), PATTERN, dtype=torch.uint8, device=DEV)
        assert raw.data_ptr() % 256 == 0
        view = raw[GUARD:GUARD + n].view(t.dtype).view(t.shape)
        view.copy_(t)
        self.raw.append((raw, n))
        return view

    def check(self):
        for i, (raw, n) in enumerate(self.raw):
            assert bool((raw[:GUARD] == PATTERN).all()), f"buffer {i}: bytes before it were written"
            tail = raw[GUARD + n:]
            assert bool((tail == PATTERN).all()), f"buffer {i}: bytes after it were written"


def _step(wl, *, window_in_pages=0, fp8=False, tuning=None, seed=None):
    stc = synth.make_structure(wl, seed)
    tokens = synth.make_tokens(stc)
    z, tokens = synth.make_logits(stc, tokens, "calibrated", conf_shift=0.3)
    q, kw, vw, kp, vp = synth.make_attn_inputs(stc)
    cfg = H.common_cfg(stc, window_in_pages=window_in_pages, s_pe=0)
    ctx = B.Context(tuning=tuning, kv_fp8=int(fp8), **cfg)
    g = Guarded()
    st = B.DeviceState.from_numpy("cpu", stc.active, stc.prefix_len, stc.L, stc.R, tokens,
                                  np.zeros((wl.n_requests, wl.wmax), np.uint8), stc.page_table)
    st = B.DeviceState(*(g.like(getattr(st, n)) for n, _ in B.fb_state._fields_))
    pk0 = B.PackBuffers.alloc(ctx, "cpu")
    pk = B.PackBuffers(*(g.like(getattr(pk0, n)) for n, _ in B.fb_pack._fields_))
    sb0 = B.StepBuffers(ctx, "cpu")
    out, argmax, conf, action, stats, ncom, spawned, ctr, status, ws = (
        g.like(getattr(sb0, n)) for n in ("out", "argmax", "conf", "action", "slot_stats", "n_committed", "spawned",
                                          "step_counters", "status", "ws"))
    dq, dkw, dvw, dz = q.to(DEV), kw.to(DEV), vw.to(DEV), z.to(DEV)
    if fp8:
        k8, v8, ks, vs = synth.make_fp8_kv(stc)
        dkp, dvp, dks, dvs = g.like(k8), g.like(v8), ks.to(DEV), vs.to(DEV)
    else:
        dkp, dvp = g.like(kp), g.like(vp)
    for _ in range(2):                                   # two steps: the second runs on the state the first left
        B.fb_pack_wavefronts(ctx, st, pk, ws, status)
        if fp8:
            B.fb_scatter_window_kv_fp8(ctx, pk, st.page_table, dkw, dvw, dkp, dvp, dks, dvs, status, rope_base=10000.0)
            B.fb_wavefront_attn_fp8(ctx, pk, dq, dkp, dvp, dks, dvs, st.page_table, out, ws, status)
        elif window_in_pages:
            B.fb_scatter_window_kv(ctx, pk, st.page_table, dkw, dvw, dkp, dvp, status, rope_base=10000.0)
            B.fb_wavefront_attn(ctx, pk, dq, None, None, dkp, dvp, st.page_table, out, ws, status)
        else:
            B.fb_wavefront_attn(ctx, pk, dq, dkw, dvw, dkp, dvp, st.page_table, out, ws, status)
        B.fb_t2t_step(ctx, pk, dz, st, argmax, conf, action, stats, status)
        resident = bool(window_in_pages)
        B.fb_gate_commit(ctx, pk, stats, st, None if resident else dkw, None if resident else dvw,
                         None if resident else dkp, None if resident else dvp, ncom, spawned, ctr, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
    g.check()


SHAPES = {
    "tiny": synth.tiny_workload(),
    "d128_w4": synth.tiny_workload(head_dim=128, n_q_heads=8, n_kv_heads=2, wmax=4, w_lo=1, w_hi=4, n_requests=6,
                                   prefix_lo=100, prefix_hi=900, max_blocks=16),
    "full_slots": synth.tiny_workload(head_dim=128, n_q_heads=8, n_kv_heads=2, wmax=3, w_lo=3, w_hi=3, n_requests=4,
                                      prefix_lo=0, prefix_hi=700, block_len=64),     # every slot live: no padding rows
}


@pytest.mark.parametrize("name", list(SHAPES))
def test_guard_bands_bf16_pages(name):
    _step(SHAPES[name])


@pytest.mark.parametrize("name", list(SHAPES))
def test_guard_bands_window_in_pages(name):
    _step(SHAPES[name], window_in_pages=1)


@pytest.mark.parametrize("name", ["d128_w4", "full_slots"])
def test_guard_bands_8_bit_pages(name):
    _step(SHAPES[name], window_in_pages=1, fp8=True)


@pytest.mark.parametrize("name", ["d128_w4", "full_slots"])
@pytest.mark.parametrize("target", [0, 100000])
def test_guard_bands_pair_kernel_and_forced_splits(name, target):
    _step(SHAPES[name], tuning=dict(attn_pair=1, attn_target_items=target))
