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
