"""Glue shared by the GPU parity tests, smoke() and the benchmark's checks:
turns one synthetic workload into (a) the oracle's Config/State and (b) the
CUDA binding's Context/DeviceState, from the same bytes.  No method arithmetic
lives here."""
from __future__ import annotations

import numpy as np
import torch

from oracle import flowblock_oracle as O
from paper_2607_17652_b200 import synth


def common_cfg(stc: synth.Structure, **over) -> dict:
    return synth.config_dict(stc, **over)


def oracle_cfg(stc, **over) -> O.Config:
    return O.Config(**common_cfg(stc, **over))


def oracle_state(stc, tokens) -> O.State:
    wl = stc.wl
    return O.State(stc.active.copy(), stc.prefix_len.copy(), stc.L.copy(),
                   stc.R.copy(), tokens.copy(),
                   np.zeros((wl.n_requests, wl.wmax), np.uint8),
                   stc.page_table.copy())


def f64(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> float64 array through the bit pattern (exact)."""
    return O.bf16_bits_to_f64(synth.to_bits(t)).reshape(t.shape)


def attn_errors(got_bf16: torch.Tensor, ref: np.ndarray, rows: np.ndarray):
    g = got_bf16.float().cpu().numpy().astype(np.float64)[rows]
    r = ref[rows]
    max_abs = float(np.abs(g - r).max()) if r.size else 0.0
    rel_l2 = float(np.linalg.norm(g - r) / max(np.linalg.norm(r), 1e-30))
    return max_abs, rel_l2


def live_rows(pk: O.Pack, b: int, slots=None) -> np.ndarray:
    if slots is None:
        return np.arange(pk.n_live * b)
    return np.concatenate([np.arange(s * b, (s + 1) * b) for s in slots])


def sub_problem(stc, tokens, attn, z_live, keep):
    """The oracle's view of a few requests of a large workload.

    ``keep``: request indices (ascending).  Builds a structure in which only
    those requests are decoding, a compact pool that holds just their pages
    (the oracle still reads every key through a page table) and the slot-order
    rows of q / k_win / v_win / logits that belong to them.  Returns a dict
    with the oracle Config/State, float64 inputs and ``rows``: the row indices
    of the FULL slot-order tensors the sub-problem's live rows correspond to.
    """
    import dataclasses
    wl = stc.wl
    b = wl.block_len
    keep = [int(r) for r in keep if stc.active[r] == 1]
    sub = dataclasses.replace(stc)
    act = np.zeros_like(stc.active)
    act[keep] = 1
    sub.active = act
    need = (stc.prefix_len + wl.wmax * b + wl.page_size - 1) // wl.page_size
    pages = np.concatenate([stc.page_table[r, :need[r]] for r in keep]) if keep else np.zeros(1, np.int32)
    remap = {int(pg): i for i, pg in enumerate(pages)}
    pt = np.zeros_like(stc.page_table)
    for r in keep:
        pt[r, :need[r]] = [remap[int(pg)] for pg in stc.page_table[r, :need[r]]]
    sub.page_table, sub.num_pages = pt, len(pages)
    ocfg = oracle_cfg(sub)
    ost = oracle_state(sub, tokens)
    full_pk = O.pack_wavefronts(oracle_cfg(stc), oracle_state(stc, tokens))
    rows = np.concatenate([np.arange(full_pk.req_slot_begin[r] * b, full_pk.req_slot_begin[r + 1] * b)
                           for r in keep]) if keep else np.zeros(0, np.int64)
    trows = torch.from_numpy(rows.astype(np.int64))
    pad = ocfg.max_slots * b - len(rows)

    def take(t):
        x = f64(t[trows])
        return np.concatenate([x, np.zeros((pad,) + x.shape[1:])], axis=0)

    out = dict(ocfg=ocfg, ost=ost, rows=rows, sub=sub)
    if attn is not None:
        q, kw, vw, kp, vp = attn
        tp = torch.from_numpy(pages.astype(np.int64))
        out.update(q=take(q), k_win=take(kw), v_win=take(vw), k_pool=f64(kp[tp]), v_pool=f64(vp[tp]))
    if z_live is not None:
        out["logits"] = take(z_live)
    return out
