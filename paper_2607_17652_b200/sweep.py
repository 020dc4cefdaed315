"""Serving sweep: requests that arrive over time, model confidences that rise
step by step, blocks that reveal, get edited, commit and spawn successors
(the staggered-arrival workload behind Sec. 4.4 / Fig. 5).

Two parts, neither of which holds any of the decode method's logic:

* :class:`SweepInputs` -- seeded inputs.  A fixed bank of N(0,1) bf16 logits,
  one row per slot-order row; every step one element per live row (the
  position's "winner" token) is overwritten so that the row's softmax
  confidence is the position's target ``c = clip(c0 + rise (step - spawn
  step), 0.02, 0.995)`` (rise = 0.05, or drawn per request), nudged until, after bf16 rounding, it is at least
  2e-3 away from both thresholds.  The confidence the patched row then has is
  returned with the patch (it follows from the bank row's sum of exponentials,
  taken once in fp64).
* :class:`SweepRunner` -- device buffers and the four calls of one step through
  the binding, timed with CUDA events.

Who decides which rows are live is the caller's business: the benchmark reads
the device state back every step, the parity test feeds the oracle's state.
"""
from __future__ import annotations

import dataclasses
import math

import numpy as np
import torch

from . import binding as B
from . import synth


def sweep_structure(wl: synth.Workload, seed: int) -> synth.Structure:
    """Every request idle, with a prompt of ``prefix`` tokens already in its
    pages and room for ``max_blocks`` generated blocks; pages scattered over
    one shared pool."""
    rg = synth._rng(seed, 7)
    Rn, b = wl.n_requests, wl.block_len
    P = rg.integers(wl.prefix_lo, wl.prefix_hi + 1, size=Rn).astype(np.int32)
    need = (P + wl.max_blocks * b + wl.page_size - 1) // wl.page_size
    maxp, total = int(need.max()), int(need.sum())
    perm = rg.permutation(total).astype(np.int32)
    pt = np.zeros((Rn, maxp), np.int32)
    off = 0
    for r in range(Rn):
        pt[r, :need[r]] = perm[off:off + need[r]]
        pt[r, need[r]:] = perm[off]
        off += need[r]
    z = np.zeros(Rn, np.int32)
    return synth.Structure(wl, seed, z.copy(), P, z.copy(), np.ones(Rn, np.int32), pt, total, maxp,
                           mask_id=wl.vocab - 1, eos_id=wl.vocab - 2)


class SweepInputs:
    def __init__(self, wl: synth.Workload, n_steps: int = 48, seed: int | None = None,
                 arrive_hi: int = 24, c_rise: float = 0.05, redraw: float = 0.1,
                 eos_frac: float = 0.25, eos_min_block: int = 8, rise_range=None):
        """``rise_range = (lo, hi)``: the per-step confidence rise is drawn per
        request from U[lo, hi] instead of being ``c_rise`` for all (easy and
        hard requests: the stragglers of a static batch)."""
        self.wl, self.n_steps = wl, n_steps
        self.seed = synth.BASE_SEED + wl.index if seed is None else seed
        self.c_rise, self.redraw = c_rise, redraw
        self.rise = np.full(wl.n_requests, c_rise)
        if rise_range is not None:
            self.rise = synth._rng(self.seed, 12).uniform(rise_range[0], rise_range[1], size=wl.n_requests)
        self.stc = sweep_structure(wl, self.seed)
        Rn, b, n, V = wl.n_requests, wl.block_len, wl.max_blocks, wl.vocab
        rg = synth._rng(self.seed, 11)
        self.arrive = rg.integers(0, max(arrive_hi, 1), size=Rn)
        self.c0 = rg.uniform(0.3, 0.9, size=(Rn, n * b))
        self.winner = rg.integers(0, V - 2, size=(Rn, n * b)).astype(np.int64)
        self.fixed = np.zeros((Rn, n * b), bool)          # positions whose winner is never re-drawn (EOS)
        if n > eos_min_block:
            for r in np.flatnonzero(rg.random(Rn) < eos_frac):
                col = int(rg.integers(eos_min_block, n)) * b + int(rg.integers(0, b))
                self.winner[r, col] = self.stc.eos_id
                self.fixed[r, col] = True
        self.winner0 = self.winner.copy()
        self.spawn_step = np.full((Rn, n), -1, np.int64)
        rows = wl.max_slots * b
        self.bank = synth.randn_bf16((rows, V), self.seed, 6)
        self.bank[:, self.stc.mask_id] = -10.0
        self.bank[:, self.stc.eos_id] = -10.0
        self.sum_exp = np.empty(rows, np.float64)         # sum_j exp(z_ij), fp64
        self.max_noise = np.empty(rows, np.float64)
        step_rows = max(1, (1 << 25) // V)
        for s in range(0, rows, step_rows):
            blk = self.bank[s:s + step_rows].to(torch.float64)
            self.sum_exp[s:s + step_rows] = torch.exp(blk).sum(1).numpy()
            self.max_noise[s:s + step_rows] = blk.max(1).values.numpy()
        self._prev = None                                  # (rows, cols) patched in the last step

    def reset(self):
        """Back to step 0 (the device copy of the bank must have been restored
        with an empty :meth:`apply` first)."""
        self.winner = self.winner0.copy()
        self.spawn_step[:] = -1
        self._prev = None

    def tokens0(self) -> np.ndarray:
        return np.full((self.wl.n_requests, self.wl.max_blocks * self.wl.block_len), self.stc.mask_id, np.int32)

    def arrivals(self, step: int):
        return [int(r) for r in np.flatnonzero(self.arrive == step)]

    def begin_step(self, step: int, active, L, R):
        """Patch list of one step for the state (active, L, R) that goes into
        it.  Returns ``(rows, cols, values, conf)``: slot-order row index,
        vocabulary column, bf16 logit (torch) and the fp64 softmax confidence
        of the patched row, for every live row."""
        wl = self.wl
        b, V = wl.block_len, wl.vocab
        rg = synth._rng(self.seed, 1000 + step)
        red = (rg.random(self.winner.shape) < self.redraw) & ~self.fixed
        new = rg.integers(0, V - 2, size=self.winner.shape)
        if step > 0:
            self.winner = np.where(red, new, self.winner)
        req, col = [], []
        for r in range(wl.n_requests):
            if active[r] != 1:
                continue
            for g in range(int(L[r]), int(R[r])):
                if self.spawn_step[r, g] < 0:
                    self.spawn_step[r, g] = step
                req.append(np.full(b, r)); col.append(g * b + np.arange(b))
        if not req:
            return (np.zeros(0, np.int64),) * 2 + (torch.zeros(0, dtype=torch.bfloat16), np.zeros(0))
        req, col = np.concatenate(req), np.concatenate(col)
        rows = np.arange(len(req))
        w = self.winner[req, col]
        c = np.clip(self.c0[req, col] + self.rise[req] * (step - self.spawn_step[req, col // b]), 0.02, 0.995)
        noise_w = self.bank[torch.from_numpy(rows), torch.from_numpy(w)].to(torch.float64).numpy()
        others = self.sum_exp[rows] - np.exp(noise_w)
        # the largest other element: the row maximum unless the winner's own noise was it
        top = self.max_noise[rows]
        thr = (float(np.float32(wl.tau_mask)), float(np.float32(wl.tau_edit)))
        a = torch.zeros(len(rows), dtype=torch.bfloat16)
        p = np.zeros(len(rows))
        todo = np.ones(len(rows), bool)
        for _ in range(200):
            idx = np.flatnonzero(todo)
            if not len(idx):
                break
            ai = torch.from_numpy(np.log(c[idx] / (1.0 - c[idx])) + np.log(others[idx])).to(torch.float32).to(torch.bfloat16)
            af = ai.to(torch.float64).numpy()
            pi = 1.0 / (1.0 + others[idx] * np.exp(-af))
            ok = (np.abs(pi - thr[0]) >= 2e-3) & (np.abs(pi - thr[1]) >= 2e-3) & (af > top[idx] + 0.05)
            a[torch.from_numpy(idx)] = ai
            p[idx] = pi
            todo[idx[ok]] = False
            bad = idx[~ok]
            c[bad] = np.where(c[bad] < 0.98, c[bad] + 0.01, c[bad] - 0.013)
        assert not todo.any(), "could not place a confidence away from the thresholds"
        return rows, w, a, p

    def apply(self, z_dev: torch.Tensor, rows, cols, values):
        """Restore last step's patched elements of the device copy of the bank
        and write this step's."""
        dev = z_dev.device
        if self._prev is not None:
            pr, pc = self._prev
            z_dev[pr.to(dev), pc.to(dev)] = self.bank[pr, pc].to(dev)
        tr, tc = torch.from_numpy(np.asarray(rows, np.int64)), torch.from_numpy(np.asarray(cols, np.int64))
        if len(tr):
            z_dev[tr.to(dev), tc.to(dev)] = values.to(dev)
        self._prev = (tr, tc)


class SweepRunner:
    """Device side of the sweep: state, pools, window tensors, the logits bank
    and the four calls of a step."""

    def __init__(self, inp: SweepInputs, device="cuda:0", window_in_pages: bool = False,
                 batch_sync: bool = False, kv_fp8: bool = False, **cfg_over):
        """``kv_fp8``: the pages hold FP8 E4M3 bytes (implies the window in the pages: the
        scatter is the quantiser)."""
        self.inp, self.dev = inp, device
        self.fp8 = bool(kv_fp8)
        self.resident = bool(window_in_pages) or self.fp8
        stc, wl = inp.stc, inp.wl
        self.ctx = B.Context(kv_fp8=int(self.fp8),
                             **synth.config_dict(stc, window_in_pages=int(self.resident),
                                                 batch_sync=int(bool(batch_sync)), **cfg_over))
        self.st = B.DeviceState.from_numpy(device, stc.active, stc.prefix_len, stc.L, stc.R, inp.tokens0(),
                                           np.zeros((wl.n_requests, wl.wmax), np.uint8), stc.page_table)
        self.pk = B.PackBuffers.alloc(self.ctx, device)
        self.sb = B.StepBuffers(self.ctx, device)
        q, kw, vw, kp, vp = synth.make_attn_inputs(stc)
        self.q, self.kw, self.vw, self.kp, self.vp = (t.to(device) for t in (q, kw, vw, kp, vp))
        if self.fp8:                     # 8-bit pools of the same N(0,1) values, per-KV-head scales
            k8, v8, ks, vs = synth.make_fp8_kv(stc)
            self.kp, self.vp, self.ks, self.vs = (t.to(device) for t in (k8, v8, ks, vs))
        self.z = inp.bank.to(device)
        self.ev = [torch.cuda.Event(enable_timing=True) for _ in range(5)]
        # written before every timed step: keeps the GPU busy while the host enqueues the
        # step (otherwise the first bracket would time the launch latency of an idle GPU,
        # not the kernel) and leaves nothing of the previous step in L2
        self.spacer = torch.empty(512 << 20, dtype=torch.uint8, device=device)

    def arrive(self, r: int):
        self.st.active[r] = 1

    def reset(self):
        """Initial state again, bank restored, inputs rewound."""
        inp, stc, wl = self.inp, self.inp.stc, self.inp.wl
        inp.apply(self.z, [], [], torch.zeros(0, dtype=torch.bfloat16))
        inp.reset()
        f = lambda t, a: t.copy_(torch.from_numpy(np.ascontiguousarray(a)).to(t.dtype))
        f(self.st.active, stc.active); f(self.st.prefix_len, stc.prefix_len)
        f(self.st.L, stc.L); f(self.st.R, stc.R); f(self.st.tokens, inp.tokens0())
        self.st.pe_done.zero_()

    def host_state(self):
        """(active, prefix_len, L, R) as they stand on the device."""
        return tuple(t.cpu().numpy() for t in (self.st.active, self.st.prefix_len, self.st.L, self.st.R))

    def step(self):
        """pack -> attention -> T2T -> gate/commit on the current stream.
        Returns the device times (ms) of the four calls."""
        ctx, st, pk, sb, ev = self.ctx, self.st, self.pk, self.sb, self.ev
        self.spacer.zero_()
        ev[0].record()
        B.fb_pack_wavefronts(ctx, st, pk, sb.ws, sb.status)
        ev[1].record()
        if self.fp8:           # Eq. 6 every step into 8-bit pages, attention with 8-bit products
            B.fb_scatter_window_kv_fp8(ctx, pk, st.page_table, self.kw, self.vw, self.kp, self.vp, self.ks, self.vs,
                                       sb.status)
            B.fb_wavefront_attn_fp8(ctx, pk, self.q, self.kp, self.vp, self.ks, self.vs, st.page_table, sb.out,
                                    sb.ws, sb.status)
        elif self.resident:    # Eq. 6 every step, attention over the pages
            B.fb_scatter_window_kv(ctx, pk, st.page_table, self.kw, self.vw, self.kp, self.vp, sb.status)
            B.fb_wavefront_attn(ctx, pk, self.q, None, None, self.kp, self.vp, st.page_table, sb.out, sb.ws,
                                sb.status)
        else:
            B.fb_wavefront_attn(ctx, pk, self.q, self.kw, self.vw, self.kp, self.vp, st.page_table, sb.out, sb.ws,
                                sb.status)
        ev[2].record()
        B.fb_t2t_step(ctx, pk, self.z, st, sb.argmax, sb.conf, sb.action, sb.slot_stats, sb.status)
        ev[3].record()
        kw, vw = (None, None) if self.resident else (self.kw, self.vw)
        B.fb_gate_commit(ctx, pk, sb.slot_stats, st, kw, vw, self.kp, self.vp, sb.n_committed,
                         sb.spawned, sb.step_counters, sb.status)
        ev[4].record()
        torch.cuda.synchronize()
        return [ev[i].elapsed_time(ev[i + 1]) for i in range(4)]
