"""Seeded synthetic inputs shaped like the paper's serving workloads.

This module only draws random numbers and lays them out; it contains none of
the method's arithmetic (no attention, no Eq. 1-3 decisions, no packing).  It
is the one module both the CUDA path's callers and the CPU oracle's callers
use, so both sides see the same bytes.  Bulk tensors are torch CPU tensors
(bf16 / int32); structure arrays are numpy.

The five workloads follow the benchmark configurations: request counts,
block length, window bound, prefix-length and live-block distributions, GQA
head counts, 64-token KV pages scattered over a shared pool, vocabulary
151,552, and the logit distributions (plain normal, "+6 winner on 70 % of
rows", and a confidence-calibrated variant that makes reveal / edit / gate
decisions actually fire).
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
import math
import numpy as np
import torch

BASE_SEED = 20260717
V_LLM = 151552


@dataclass(frozen=True)
class Workload:
    name: str
    index: int
    n_requests: int
    block_len: int
    wmax: int
    prefix_lo: int
    prefix_hi: int
    w_lo: int
    w_hi: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    vocab: int
    logits_kind: str            # "normal2" | "literal" | "calibrated"
    mask_mode: str              # "half" | "uniform_fraction"
    max_blocks: int = 64
    page_size: int = 64
    tau_mask: float = 0.9
    tau_edit: float = 0.95
    theta_spawn: float = 0.5
    s_pe: int = 1

    @property
    def max_slots(self):
        return self.n_requests * self.wmax


WORKLOADS = {
    0: Workload("cfg0_single_request", 0, 1, 32, 2, 64, 64, 2, 2, 4, 1, 64,
                1024, "normal2", "half", max_blocks=8),
    1: Workload("cfg1_batch8", 1, 8, 32, 4, 256, 2048, 1, 4, 16, 4, 128,
                V_LLM, "literal", "half"),
    2: Workload("cfg2_batch64", 2, 64, 32, 4, 1024, 8192, 1, 4, 32, 8, 128,
                V_LLM, "literal", "uniform_fraction"),
    3: Workload("cfg3_longctx16", 3, 16, 64, 3, 16384, 32768, 3, 3, 32, 8,
                128, V_LLM, "literal", "half", max_blocks=32),
    4: Workload("cfg4_serving128", 4, 128, 32, 4, 512, 4096, 1, 4, 32, 8,
                128, V_LLM, "calibrated", "uniform_fraction"),
}


def tiny_workload(**kw) -> Workload:
    """A small workload for element-by-element parity (several tiles and a
    ragged tail, but seconds for the oracle)."""
    base = Workload("tiny", 99, 3, 32, 3, 5, 300, 1, 3, 8, 2, 64, 512,
                    "calibrated", "uniform_fraction", max_blocks=12)
    return replace(base, **kw)


def _rng(seed, stream):
    return np.random.Generator(np.random.Philox(key=[seed & 0xFFFFFFFF, stream]))


def _tgen(seed, stream):
    g = torch.Generator(device="cpu")
    g.manual_seed((seed * 1000003 + stream) & 0x7FFFFFFFFFFFFFFF)
    return g


@dataclass
class Structure:
    wl: Workload
    seed: int
    active: np.ndarray
    prefix_len: np.ndarray
    L: np.ndarray
    R: np.ndarray
    page_table: np.ndarray
    num_pages: int
    max_pages_per_req: int
    mask_id: int
    eos_id: int


def make_structure(wl: Workload, seed: int | None = None, n_inactive: int = 0,
                   scatter_pages: bool = True) -> Structure:
    """Per-request prefix lengths, live-block counts and a page table whose
    pages are a random permutation of one shared pool.  ``n_inactive``
    requests (chosen at random) are left free (active = 0)."""
    seed = BASE_SEED + wl.index if seed is None else seed
    rg = _rng(seed, 7)
    Rn, b = wl.n_requests, wl.block_len
    P = rg.integers(wl.prefix_lo, wl.prefix_hi + 1, size=Rn).astype(np.int32)
    Wr = rg.integers(wl.w_lo, wl.w_hi + 1, size=Rn).astype(np.int32)
    # blocks committed so far: part of the prefix is earlier generation
    Lr = np.minimum(P // b, rg.integers(0, 9, size=Rn)).astype(np.int32)
    Lr = np.minimum(Lr, wl.max_blocks - Wr).astype(np.int32)
    Rr = (Lr + Wr).astype(np.int32)
    active = np.ones(Rn, np.int32)
    if n_inactive:
        active[rg.choice(Rn, size=n_inactive, replace=False)] = 0
    need = (P + wl.wmax * b + wl.page_size - 1) // wl.page_size
    maxp = int(need.max())
    total = int(need.sum())
    perm = rg.permutation(total).astype(np.int32) if scatter_pages \
        else np.arange(total, dtype=np.int32)
    pt = np.zeros((Rn, maxp), np.int32)
    off = 0
    for r in range(Rn):
        pt[r, :need[r]] = perm[off:off + need[r]]
        pt[r, need[r]:] = perm[off]          # any valid page id
        off += need[r]
    return Structure(wl, seed, active, P, Lr, Rr, pt, total, maxp,
                     mask_id=wl.vocab - 1, eos_id=wl.vocab - 2)


def config_dict(stc: Structure, **over) -> dict:
    """The fb_config / oracle Config fields of a workload, as keyword args."""
    wl = stc.wl
    d = dict(max_requests=wl.n_requests, wmax=wl.wmax, block_len=wl.block_len,
             n_q_heads=wl.n_q_heads, n_kv_heads=wl.n_kv_heads,
             head_dim=wl.head_dim, page_size=wl.page_size,
             num_pages=stc.num_pages, max_pages_per_req=stc.max_pages_per_req,
             vocab=wl.vocab, mask_id=stc.mask_id, eos_id=stc.eos_id,
             max_blocks=wl.max_blocks, s_pe=wl.s_pe, tau_mask=wl.tau_mask,
             tau_edit=wl.tau_edit, theta_spawn=wl.theta_spawn, sm_scale=0.0)
    d.update(over)
    return d


def n_live_slots(stc: Structure) -> int:
    return int(((stc.R - stc.L) * (stc.active == 1)).sum())


def make_tokens(stc: Structure) -> np.ndarray:
    """tokens [R, n*bl]: committed blocks hold token ids, live blocks hold a
    mix of [M] and token ids (exact count per block, positions by seeded
    shuffle), blocks to the right are all [M]."""
    wl = stc.wl
    rg = _rng(stc.seed, 8)
    b = wl.block_len
    tok = np.full((wl.n_requests, wl.max_blocks * b), stc.mask_id, np.int32)
    for r in range(wl.n_requests):
        for g in range(int(stc.R[r])):
            ids = rg.integers(0, wl.vocab - 2, size=b)
            if g >= stc.L[r]:
                if wl.mask_mode == "half":
                    nm = b // 2
                else:
                    nm = int(round(rg.uniform(0.0, 1.0) * b))
                ids[rg.permutation(b)[:nm]] = stc.mask_id
            tok[r, g * b:(g + 1) * b] = ids
    return tok


def randn_bf16(shape, seed, stream, std=1.0) -> torch.Tensor:
    """N(0, std^2) rounded to bf16 (round-to-nearest-even)."""
    n = int(np.prod(shape))
    out = torch.empty(n, dtype=torch.bfloat16)
    g = _tgen(seed, stream)
    chunk = 1 << 24
    for s in range(0, n, chunk):
        e = min(n, s + chunk)
        x = torch.randn(e - s, generator=g, dtype=torch.float32)
        if std != 1.0:
            x.mul_(std)
        out[s:e] = x.to(torch.bfloat16)
    return out.view(*shape)


def make_attn_inputs(stc: Structure, fill_unused: float | None = None):
    """Q, window K/V in slot order and the paged prefix pools, N(0,1) bf16.
    Rows of padding slots and never-visible pool positions are random too
    (finite), so a kernel that reads them by mistake shows up as an error."""
    wl = stc.wl
    S, b = wl.max_slots, wl.block_len
    q = randn_bf16((S * b, wl.n_q_heads, wl.head_dim), stc.seed, 1)
    k_win = randn_bf16((S * b, wl.n_kv_heads, wl.head_dim), stc.seed, 2)
    v_win = randn_bf16((S * b, wl.n_kv_heads, wl.head_dim), stc.seed, 3)
    shape = (stc.num_pages, wl.n_kv_heads, wl.page_size, wl.head_dim)
    k_pool = randn_bf16(shape, stc.seed, 4)
    v_pool = randn_bf16(shape, stc.seed, 5)
    return q, k_win, v_win, k_pool, v_pool


def make_fp8_kv(stc: Structure, amax: float = 6.0):
    """8-bit KV pools for the FP8-page variant: per-KV-head scales (what a
    calibration pass would hand over: ``amax`` standard deviations of N(0,1)
    map to the top of the E4M3 range, times a per-head factor in [0.5, 2] so
    that heads differ) and pools of random E4M3 bytes, drawn as N(0,1) / scale
    and cast with the library's float8 type.  Returns (k_pool8, v_pool8) uint8
    [num_pages, Hkv, page, d] and (k_scale, v_scale) float32 [Hkv]."""
    wl = stc.wl
    rg = _rng(stc.seed, 15)
    ks = (amax / 448.0 * rg.uniform(0.5, 2.0, size=wl.n_kv_heads)).astype(np.float32)
    vs = (amax / 448.0 * rg.uniform(0.5, 2.0, size=wl.n_kv_heads)).astype(np.float32)
    shape = (stc.num_pages, wl.n_kv_heads, wl.page_size, wl.head_dim)
    pools = []
    for stream, sc in ((4, ks), (5, vs)):
        x = randn_bf16(shape, stc.seed, stream).to(torch.float32)
        x = (x / torch.from_numpy(sc)[None, :, None, None]).clamp_(-448.0, 448.0)
        pools.append(x.to(torch.float8_e4m3fn).view(torch.uint8))
    return pools[0], pools[1], torch.from_numpy(ks), torch.from_numpy(vs)


def _slot_rows(stc: Structure):
    """(request, block, token) of every live row in slot order -- plain
    enumeration of live blocks, used only to place winners and tokens."""
    wl = stc.wl
    rows = []
    for r in range(wl.n_requests):
        if stc.active[r] != 1:
            continue
        for g in range(int(stc.L[r]), int(stc.R[r])):
            for t in range(wl.block_len):
                rows.append((r, g, t))
    return rows


def make_logits(stc: Structure, tokens: np.ndarray, kind: str | None = None,
                seed_shift: int = 0, conf_shift: float = 0.0,
                n_rows: int | None = None):
    """bf16 logits [max_slots*bl, V] in slot order, plus the (possibly
    adjusted) tokens.

    kind "normal2":    N(0, variance 2).
    kind "literal":    N(0,1); on 70 % of rows one uniformly drawn token gets
                       +6 before rounding.
    kind "calibrated": N(0,1); on 70 % of live rows the winner's logit is set
                       so that its softmax confidence is c ~ U(0.5, 0.999)
                       (+ conf_shift), nudged until, after bf16 rounding, the
                       confidence is at least 2e-3 away from tau_mask and
                       tau_edit; 30 % of those rows at revealed positions get
                       a current token different from the winner (so edits
                       fire), the rest get the winner as current token.
    The [M] and EOS columns are set to -10 so that neither is ever the top-1
    token by accident."""
    wl = stc.wl
    kind = kind or wl.logits_kind
    V, b = wl.vocab, wl.block_len
    rows_total = wl.max_slots * b if n_rows is None else n_rows
    seed = stc.seed + 7919 * seed_shift
    std = math.sqrt(2.0) if kind == "normal2" else 1.0
    z = randn_bf16((rows_total, V), seed, 6, std)
    z[:, stc.mask_id] = -10.0
    z[:, stc.eos_id] = -10.0
    tokens = tokens.copy()
    if kind == "normal2":
        return z, tokens
    rg = _rng(seed, 9)
    live = _slot_rows(stc)
    n_live_rows = min(len(live), rows_total)
    pick = rg.random(rows_total) < 0.7
    winners = rg.integers(0, V - 2, size=rows_total)
    if kind == "literal":
        idx = np.flatnonzero(pick)
        zi = z[idx, winners[idx]].to(torch.float32) + 6.0
        z[idx, winners[idx]] = zi.to(torch.bfloat16)
        return z, tokens
    assert kind == "calibrated"
    cs = np.clip(rg.uniform(0.5, 0.999, size=rows_total) + conf_shift,
                 0.02, 0.9995)
    flip = rg.random(rows_total) < 0.3
    thr = (float(np.float32(wl.tau_mask)), float(np.float32(wl.tau_edit)))
    for i in range(n_live_rows):
        if not pick[i]:
            continue
        w = int(winners[i])
        row = z[i].to(torch.float64)
        row[w] = -float("inf")
        lse = float(torch.logsumexp(row, 0))
        c = float(cs[i])
        for _ in range(200):
            a = torch.tensor(math.log(c / (1.0 - c)) + lse,
                             dtype=torch.float32).to(torch.bfloat16)
            p = 1.0 / (1.0 + math.exp(lse - float(a)))
            if all(abs(p - t) >= 2e-3 for t in thr) and float(a) > float(row.max()) + 0.05:
                break
            c = min(0.9995, c + 0.01) if c < 0.99 else c - 0.013
        z[i, w] = a
        r, g, t = live[i]
        col = g * b + t
        if tokens[r, col] != stc.mask_id:
            tokens[r, col] = (w + 1) % (V - 2) if flip[i] else w
    return z, tokens


def to_bits(t: torch.Tensor) -> np.ndarray:
    """bf16 torch tensor -> uint16 bit patterns (numpy, no copy of meaning)."""
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def make_lm_head_inputs(stc: Structure, tokens: np.ndarray, hidden: int,
                        seed_shift: int = 0):
    """Hidden states x [max_slots*bl, hidden] and LM-head weights w [V, hidden]
    (bf16) whose logits x w^T look like the "calibrated" logits of
    :func:`make_logits`: N(0,1) noise, and on 70 % of the live rows a winner
    token whose softmax confidence is c ~ U(0.5, 0.999), placed by moving the
    row's hidden state along the winner's weight vector and nudged until, for
    the bf16-rounded inputs, the confidence is at least 2e-3 away from tau_mask
    and tau_edit and the winner leads by 0.05.  Revealed positions get the
    winner or (30 %) another token as current token.  The [M] and EOS rows of
    w are zero.  Returns (x, w, tokens)."""
    wl = stc.wl
    V, b = wl.vocab, wl.block_len
    rows = wl.max_slots * b
    seed = stc.seed + 7919 * seed_shift
    w = randn_bf16((V, hidden), seed, 13, 1.0 / math.sqrt(hidden))
    w[stc.mask_id] = 0.0
    w[stc.eos_id] = 0.0
    x = randn_bf16((rows, hidden), seed, 14)
    tokens = tokens.copy()
    rg = _rng(seed, 15)
    live = _slot_rows(stc)
    pick = rg.random(rows) < 0.7
    winners = rg.integers(0, V - 2, size=rows)
    cs = rg.uniform(0.5, 0.999, size=rows)
    flip = rg.random(rows) < 0.3
    thr = (float(np.float32(wl.tau_mask)), float(np.float32(wl.tau_edit)))
    w64 = w.to(torch.float64)
    for i in range(min(len(live), rows)):
        if not pick[i]:
            continue
        wi = int(winners[i])
        dirv = w64[wi] / float(w64[wi] @ w64[wi])            # moves z_w by 1 per unit
        xi = x[i].to(torch.float64)
        c = float(cs[i])
        for _ in range(300):
            z = w64 @ xi
            zo = z.clone()
            zo[wi] = -float("inf")
            want = math.log(c / (1.0 - c)) + float(torch.logsumexp(zo, 0))
            cand = (xi + (want - float(z[wi])) * dirv).to(torch.bfloat16).to(torch.float64)
            z = w64 @ cand
            zo = z.clone()
            zo[wi] = -float("inf")
            p = 1.0 / (1.0 + math.exp(float(torch.logsumexp(zo, 0)) - float(z[wi])))
            if all(abs(p - t) >= 2e-3 for t in thr) and float(z[wi]) > float(zo.max()) + 0.05:
                x[i] = cand.to(torch.bfloat16)
                break
            c = min(0.9995, c + 0.01) if c < 0.99 else c - 0.013
        else:
            raise RuntimeError("could not place a confidence away from the thresholds")
        r, g, t = live[i]
        col = g * b + t
        if tokens[r, col] != stc.mask_id:
            tokens[r, col] = (wi + 1) % (V - 2) if flip[i] else wi
    return x, w, tokens
