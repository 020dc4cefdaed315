"""Plain fp64 CPU oracle for one packed FlowBlock decode step.

THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  Only the test-suite, the smoke
check and the CPU-baseline leg of the benchmark may import it.  It shares no
code with the CUDA path and never imports the CUDA package; the CUDA package
never imports it.

Everything here is the definition written out with straight loops and numpy
fp64 primitives (a matmul, a max, an exp) -- no tiling, no online softmax, no
fusion -- so that each function can be checked against the paper by eye.

Notation (the paper's): requests b (here index r), block length bl (here
``b``), window [L, R) of at most W adjacent live blocks, absolute offset
o_b = start(B_L) (here ``prefix_len`` P_r, the number of frozen-prefix
tokens = prompt + committed blocks), thresholds tau_mask, tau_edit,
theta_spawn, post-edit budget S_pe.

Pins (tests/test_oracle_*.py, all CPU):
  pack_wavefronts        brute-force enumeration on random states; q = W*bl
                         worked value of the Discussion paragraph (Sec. 3.2)
  wavefront_attn         literal dense-mask attention in the paper's physical
                         layout (Eq. 5) on tiny inputs; closed forms (zero
                         query -> mean of visible V rows; constant V; one
                         dominant key); isolation; block causality
  t2t_rows               closed form e^a / (e^a + V - 1); ties -> lowest index
  t2t_update             hand-worked Eq. 1 / Eq. 2 case; literal Delta: hand-worked
                         rows, and no effect when tau_edit >= tau_mask; forced
                         progress: hand-worked block, no effect where Eq. 1
                         reveals something, termination within bl + S_pe + 1
                         steps per block on logits that never clear a threshold
  gate_commit            hand-worked Alg. 1 cases; window of one block equals
                         an independently written serial block-wise decoder;
                         packed run equals per-request runs
  gate_commit_batch_sync one sequence: equal to gate_commit (Sec. 4.5: "at
                         B = 1 the two are semantically identical"); copies of
                         one sequence: equal to gate_commit; hand-worked
                         straggler, EOS and min-rho cases; lockstep invariant
  scatter_window_kv      brute-force placement (every live window position, no
                         other pool element); attention over the page-resident
                         window equals attention over the slot-order window;
                         pointer-bump commit equals copy-at-commit
  embed_gather           brute force over (request, block, token)
  lm_head_rows           one-hot hidden states read the closed-form rows of
                         t2t_rows back out of the weights; scaling x scales
                         the logits; permuting the vocabulary permutes argmax
  rope_rotate            textbook special cases (position 0, d = 2 rotation,
                         norm, relative-offset invariance of q.k)
  e4m3_decode / e4m3_quantize
                         all 256 codes against the format's closed form and
                         against a library conversion; round trip of every
                         finite code; hand-worked ties, subnormals, saturation;
                         monotonicity; power-of-two scale invariance
  scatter_window_kv_fp8 / wavefront_attn_fp8
                         placement as scatter_window_kv; with representable
                         values and scale 1 both reduce to the bf16-path
                         functions exactly; dequantised error <= half a code
                         step; scale folded into the scores / the output
Nothing in this file is "parity unpinned".

Readings of the paper taken where it is silent or ambiguous are the named
constants / comments marked READING below.
"""
from __future__ import annotations

from dataclasses import dataclass, field
import numpy as np

FLAG_OLDEST = 1     # slot is block L of its request (leftmost, next to commit)
FLAG_FRONTIER = 2   # slot is block R-1 of its request (readiness is read here)

ACT_NONE = 0
ACT_M2T = 1         # masked position revealed (set Gamma of Eq. 1)
ACT_T2T = 2         # revealed position overwritten (set Delta of Eq. 1)
ACT_FORCED = 3      # masked position revealed by the forced-progress rule

# slot_stats columns
ST_M0, ST_RDY, ST_M2T, ST_T2T, ST_M1, ST_EOS = range(6)
# step_counters entries
(CT_BLOCKS, CT_TOKENS, CT_SPAWNED, CT_FINISHED, CT_M2T, CT_T2T,
 CT_LIVE_SLOTS, CT_ACTIVE, CT_LOCKSTEP_COMMIT, CT_LOCKSTEP_ADMIT) = range(10)
N_COUNTERS = 10


@dataclass
class Config:
    max_requests: int
    wmax: int                 # W, window bound (Sec. 3.1, "Wavefront window")
    block_len: int            # bl
    n_q_heads: int = 1
    n_kv_heads: int = 1
    head_dim: int = 8
    page_size: int = 64
    num_pages: int = 0
    max_pages_per_req: int = 0
    vocab: int = 4
    mask_id: int = 4
    eos_id: int = -1
    max_blocks: int = 1       # n, number of generation blocks (Alg. 1 REQUIRE)
    s_pe: int = 1             # S_pe (Sec. 2.1); READING: value never given
    tau_mask: float = 0.9
    tau_edit: float = 0.95
    theta_spawn: float = 0.5
    sm_scale: float = 0.0     # 0 -> 1/sqrt(head_dim); READING: paper silent
    batch_sync: int = 0       # 1: the batch-synchronous wavefront of Sec. 3.2 / 4.5
    delta_literal: int = 0    # 1: Delta of Eq. 1 as printed (masked positions too)
    force_progress: int = 0   # 1: the oldest block reveals at least one mask per step

    @property
    def max_slots(self) -> int:
        return self.max_requests * self.wmax

    @property
    def q_capacity(self) -> int:
        """q = W * bl, the fixed per-window capacity (Sec. 3.2, Eq. 4)."""
        return self.wmax * self.block_len


@dataclass
class State:
    """Per-request wavefront state (Sec. 3.2: (L_b, R_b), finished flags,
    in-order commit pointer).  All arrays are modified in place by the step."""
    active: np.ndarray        # int32 [R]  0 free, 1 decoding, 2 done
    prefix_len: np.ndarray    # int32 [R]  o_b: tokens in the frozen prefix
    L: np.ndarray             # int32 [R]
    R: np.ndarray             # int32 [R]
    tokens: np.ndarray        # int32 [R, n*bl] generation region, mask_id=[M]
    pe_done: np.ndarray       # uint8 [R, W] post-edit forwards seen per slot
    page_table: np.ndarray    # int32 [R, max_pages_per_req]

    def copy(self) -> "State":
        return State(*(getattr(self, f).copy() for f in
                       ("active", "prefix_len", "L", "R", "tokens",
                        "pe_done", "page_table")))


@dataclass
class Pack:
    n_live: int
    slot_req: np.ndarray
    slot_s: np.ndarray
    slot_pos0: np.ndarray
    slot_kv_len: np.ndarray
    slot_flags: np.ndarray
    req_slot_begin: np.ndarray
    qtok: np.ndarray
    pos: np.ndarray


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bfloat16 bit patterns (uint16) to float64."""
    u = np.asarray(bits).view(np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


# --------------------------------------------------------------------------
# a1  pack: per-request states -> dense slot batch   (Sec. 3.2, Eq. 4)
# --------------------------------------------------------------------------
def pack_wavefronts(cfg: Config, st: State) -> Pack:
    """Gather of Eq. 4 over live blocks only.

    Every decoding request r contributes its W_r = R_r - L_r live blocks as
    consecutive slots, requests in index order, blocks left to right.  Slot
    (r, s) holds tokens x[r, o_r + s*bl + [0..bl)) and absolute position ids
    o_r + s*bl + [0..bl)  (Eq. 4 with o_b = prefix_len[r]; ``tokens`` stores
    the generation region, so block g starts at column g*bl).
    READING: the paper forwards all q = W*bl positions of every window; here
    only admitted blocks become slots and the batch is padded to the fixed
    max_slots = max_requests * W (shape stability, Sec. 3.2), padding slots
    carrying req = -1, qtok = mask_id, pos = 0.
    kv_len = o_r + (s+1)*bl is the number of keys the slot may see (Eq. 5).
    """
    b, S = cfg.block_len, cfg.max_slots
    slot_req = np.full(S, -1, np.int32)
    slot_s = np.zeros(S, np.int32)
    slot_pos0 = np.zeros(S, np.int32)
    slot_kv_len = np.zeros(S, np.int32)
    slot_flags = np.zeros(S, np.int32)
    begin = np.zeros(cfg.max_requests + 1, np.int32)
    qtok = np.full(S * b, cfg.mask_id, np.int32)
    pos = np.zeros(S * b, np.int32)
    n = 0
    for r in range(cfg.max_requests):
        begin[r] = n
        if st.active[r] != 1:
            continue
        w = int(st.R[r]) - int(st.L[r])
        for s in range(w):
            g = int(st.L[r]) + s
            slot_req[n] = r
            slot_s[n] = s
            slot_pos0[n] = st.prefix_len[r] + s * b
            slot_kv_len[n] = st.prefix_len[r] + (s + 1) * b
            slot_flags[n] = (FLAG_OLDEST if s == 0 else 0) | \
                            (FLAG_FRONTIER if s == w - 1 else 0)
            for t in range(b):
                qtok[n * b + t] = st.tokens[r, g * b + t]
                pos[n * b + t] = slot_pos0[n] + t
            n += 1
    begin[cfg.max_requests] = n
    return Pack(n, slot_req, slot_s, slot_pos0, slot_kv_len, slot_flags,
                begin, qtok, pos)


# --------------------------------------------------------------------------
# a2  W-shaped block-causal attention   (Sec. 3.1 "W-shaped block-causal
#     attention"; Sec. 3.2 Eq. 5)
# --------------------------------------------------------------------------
def _scale(cfg: Config) -> float:
    return cfg.sm_scale if cfg.sm_scale != 0.0 else 1.0 / np.sqrt(cfg.head_dim)


def visible_keys(cfg: Config, pk: Pack, slot: int, k_win, k_pool, page_table):
    """Rows of K (or V) visible to the queries of ``slot``, for all KV heads:
    the request's committed prefix [0, o_r) read through its page table, then
    window blocks L..g of the same request (g = the slot's own block), every
    token of each -- bidirectional inside a block, nothing to the right.
    With ``k_win`` None the window is resident in the pages as well (it was
    scattered there, Eq. 6) and every key is read through the page table.
    Returns [kv_len, Hkv, d]."""
    b, ps = cfg.block_len, cfg.page_size
    r, s = int(pk.slot_req[slot]), int(pk.slot_s[slot])
    first = int(pk.req_slot_begin[r])
    P = int(pk.slot_pos0[slot]) - s * b
    rows = []
    for j in range(P if k_win is not None else P + (s + 1) * b):
        page = int(page_table[r, j // ps])
        rows.append(k_pool[page, :, j % ps, :])
    for s2 in range(s + 1 if k_win is not None else 0):
        for t in range(b):
            rows.append(k_win[(first + s2) * b + t])
    return np.stack(rows, axis=0)


def wavefront_attn(cfg: Config, pk: Pack, q, k_win, v_win, k_pool, v_pool,
                   page_table, only_slots=None) -> np.ndarray:
    """Softmax attention of every live query over its visible keys.

    q [S*bl, Hq, d]; k_win, v_win [S*bl, Hkv, d] (slot order, this step's
    fresh window K/V); k_pool, v_pool [num_pages, Hkv, page, d]; all float64.
    Query head h uses KV head h // (Hq/Hkv).  Masked keys are excluded
    outright (READING: -inf, never a finite fill); scale 1/sqrt(d) unless
    given.  Two-pass softmax in fp64.  Padding-slot rows are returned as 0.
    ``only_slots`` restricts the computation to a subset of live slots (the
    other rows stay 0); used for sampled checks at large sizes.
    """
    b, Hq, Hkv, d = cfg.block_len, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    G = Hq // Hkv
    sc = _scale(cfg)
    out = np.zeros((cfg.max_slots * b, Hq, d), np.float64)
    for slot in (range(pk.n_live) if only_slots is None else only_slots):
        K = visible_keys(cfg, pk, slot, k_win, k_pool, page_table)
        V = visible_keys(cfg, pk, slot, v_win, v_pool, page_table)
        for h in range(Hq):
            kh = h // G
            Q = q[slot * b:(slot + 1) * b, h, :]            # [bl, d]
            sco = sc * (Q @ K[:, kh, :].T)                  # [bl, kv_len]
            m = sco.max(axis=1, keepdims=True)
            w = np.exp(sco - m)
            out[slot * b:(slot + 1) * b, h, :] = \
                (w @ V[:, kh, :]) / w.sum(axis=1, keepdims=True)
    return out


def wavefront_attn_weight_norms(cfg: Config, pk: Pack, q, k_win, k_pool, page_table) -> np.ndarray:
    """sum_i w_i^2 of the softmax weights of every live query row and head,
    [S*bl, Hq] (1/n for n equal weights, 1 when one key takes everything).  Not
    part of the method: the tests of approximate kernels scale their
    element-wise error bounds with it (independent per-weight errors of relative
    size eps leave eps * sqrt(sum w_i^2) * rms(v) in an output element)."""
    b, Hq, Hkv = cfg.block_len, cfg.n_q_heads, cfg.n_kv_heads
    G = Hq // Hkv
    sc = _scale(cfg)
    out = np.zeros((cfg.max_slots * b, Hq), np.float64)
    for slot in range(pk.n_live):
        K = visible_keys(cfg, pk, slot, k_win, k_pool, page_table)
        for h in range(Hq):
            sco = sc * (q[slot * b:(slot + 1) * b, h, :] @ K[:, h // G, :].T)
            w = np.exp(sco - sco.max(axis=1, keepdims=True))
            w = w / w.sum(axis=1, keepdims=True)
            out[slot * b:(slot + 1) * b, h] = (w * w).sum(axis=1)
    return out


def dense_mask_attn_bruteforce(cfg: Config, st_prefix_len, st_wlive, q_req,
                               k_phys, v_phys, C: int) -> np.ndarray:
    """Literal Eq. 5 in the paper's own physical layout, for tiny sizes.

    Row b of the batch owns a cache of C positions: its frozen prefix at
    [0, o_b), anything at all in the stale middle [o_b, t), and the window at
    the shared physical tail [t, t+q), t = C - q, q = W*bl.  Query i of the
    window (slot s = floor(i/bl)) may see j iff  j < o_b  or
    t <= j < t + (s+1)*bl.  The mask is built as a dense boolean array and
    applied to a dense score matrix.
      q_req  [B, q, Hq, d]   k_phys, v_phys [B, C, Hkv, d]
    Returns [B, q, Hq, d]; rows of un-admitted window blocks are computed too
    (the caller ignores them)."""
    B = len(st_prefix_len)
    bl, W = cfg.block_len, cfg.wmax
    qcap = W * bl
    t = C - qcap
    G = cfg.n_q_heads // cfg.n_kv_heads
    sc = _scale(cfg)
    out = np.zeros_like(q_req)
    for bi in range(B):
        o = int(st_prefix_len[bi])
        assert o <= t
        M = np.zeros((qcap, C), bool)
        for i in range(qcap):
            s = i // bl
            for j in range(C):
                M[i, j] = (j < o) or (t <= j < t + (s + 1) * bl)
        for h in range(cfg.n_q_heads):
            S_ = sc * (q_req[bi, :, h, :] @ k_phys[bi, :, h // G, :].T)
            S_ = np.where(M, S_, -np.inf)
            S_ = S_ - S_.max(axis=1, keepdims=True)
            Pm = np.exp(S_)
            Pm = Pm / Pm.sum(axis=1, keepdims=True)
            out[bi, :, h, :] = Pm @ v_phys[bi, :, h // G, :]
    return out


# --------------------------------------------------------------------------
# next: Eq. 6 as data movement -- the window resident in the pages
# --------------------------------------------------------------------------
def rope_rotate(x, pos, base: float):
    """Rotary position embedding of one vector (last axis = head dim d) at
    absolute position ``pos``: pair (x_i, x_{i+d/2}), i < d/2, is rotated by the
    angle pos * base^(-2i/d).

    READING: the paper only says that the gathered window carries "absolute
    position ids for RoPE" (Sec. 3.2); the pairing (rotate-half) and the base
    are the model's, taken here as parameters."""
    d = x.shape[-1]
    i = np.arange(d // 2, dtype=np.float64)
    ang = float(pos) * np.power(float(base), -2.0 * i / d)
    c, s = np.cos(ang), np.sin(ang)
    lo, hi = x[..., :d // 2], x[..., d // 2:]
    return np.concatenate([lo * c - hi * s, hi * c + lo * s], axis=-1)


def scatter_window_kv(cfg: Config, pk: Pack, k_new, v_new, k_pool, v_pool,
                      page_table, rope_base: float = 0.0):
    """Eq. 6 as data movement: the fresh K/V of every live window position go
    to the request's pages at their absolute positions, cache[r, o_r + s*bl +
    t] = k_new[slot, t], every step; in place on the pools.

    k_new, v_new [S*bl, Hkv, d] in slot order.  With ``rope_base`` > 0 the keys
    are rotated by their absolute position first (rope_rotate); V never is.
    The frozen prefix [0, o_r) and every position right of the window are not
    touched.  Retirement then needs no copy: advancing o_r freezes what is
    already in place."""
    b, ps = cfg.block_len, cfg.page_size
    for slot in range(pk.n_live):
        r = int(pk.slot_req[slot])
        for t in range(b):
            pos = int(pk.slot_pos0[slot]) + t
            page = int(page_table[r, pos // ps])
            k = k_new[slot * b + t]
            if rope_base > 0.0:
                k = rope_rotate(k, pos, rope_base)
            k_pool[page, :, pos % ps, :] = k
            v_pool[page, :, pos % ps, :] = v_new[slot * b + t]


# --------------------------------------------------------------------------
# next: the KV pages held in 8 bits (FP8 E4M3)
# --------------------------------------------------------------------------
# READING (the paper states no numeric precision, Sec. 4.1; the cache is the
# one Sec. 3.2 "KV Retrieval and Write-back" / Eq. 6 defines): a page stores
# K and V as OCP FP8 E4M3 codes (1 sign, 4 exponent bits with bias 7, 3 mantissa
# bits; no infinities, S.1111.111 is NaN, largest finite value 448) with one
# binary32 scale per KV head for K and one for V, given by the caller:
# stored code = e4m3(x / scale), value read back = code * scale.  One scale per
# head and not per page, because a 64-token page is filled by several commits
# of bl-token blocks and a per-page scale would have to re-quantise positions
# that are already frozen (Sec. 3.1: a committed block's KV is exact and never
# rewritten).  Where rounding decides the stored byte it is taken in binary32,
# the precision the writer computes in: x / scale as a correctly rounded
# binary32 quotient, then round-to-nearest-even onto the E4M3 grid, saturating
# at +-448.
E4M3_MAX = 448.0


def e4m3_decode(codes) -> np.ndarray:
    """Value of each E4M3 code (uint8 array) as float64: (-1)^s 2^(e-7) (1 + m/8)
    for e > 0, (-1)^s 2^-6 (m/8) for e = 0; the two NaN codes give NaN."""
    c = np.asarray(codes, np.uint8).astype(np.int64)
    sgn = np.where(c & 0x80, -1.0, 1.0)
    e = (c >> 3) & 0xF
    m = (c & 7).astype(np.float64)
    val = np.where(e > 0, np.ldexp(1.0 + m / 8.0, e - 7), np.ldexp(m / 8.0, -6))
    val = sgn * val
    return np.where((c & 0x7F) == 0x7F, np.nan, val)


def e4m3_round(y) -> np.ndarray:
    """Codes of the E4M3 values nearest to the finite numbers ``y`` (ties to
    the even mantissa, magnitudes beyond 448 saturate to 448)."""
    y = np.asarray(y, np.float64)
    a = np.minimum(np.abs(y), E4M3_MAX)
    # spacing of the grid around a: 2^(floor(log2 a) - 3) for normal values, 2^-9 below 2^-6
    ex = np.floor(np.log2(np.maximum(a, 2.0 ** -6)))
    step = np.exp2(ex - 3)
    n = np.rint(a / step)                      # numpy rounds halves to even; a / step is exact (power of two)
    v = n * step                               # may have carried into the next binade: still on the grid
    e = np.floor(np.log2(np.maximum(v, 2.0 ** -6)))
    is_sub = v < 2.0 ** -6
    mant = np.where(is_sub, v / 2.0 ** -9, v / np.exp2(e - 3) - 8.0)
    code = np.where(is_sub, mant, (e + 7) * 8 + mant).astype(np.int64)
    code = np.where(np.signbit(y), code | 0x80, code)
    return code.astype(np.uint8)


def e4m3_quantize(x, scale) -> np.ndarray:
    """Stored bytes of values ``x`` under ``scale`` (broadcast): the binary32
    quotient x / scale rounded to E4M3."""
    quot = (np.asarray(x, np.float64).astype(np.float32) / np.asarray(scale, np.float32)).astype(np.float64)
    return e4m3_round(quot)


def scatter_window_kv_fp8(cfg: Config, pk: Pack, k_new, v_new, k_pool8,
                          v_pool8, k_scale, v_scale, page_table,
                          rope_base: float = 0.0):
    """scatter_window_kv into 8-bit pages: the (optionally rotated) fresh K/V
    of every live window position are quantised with their KV head's scale and
    stored at their absolute positions; in place on the uint8 pools
    [num_pages, Hkv, page, d].  k_scale, v_scale [Hkv]."""
    b, ps = cfg.block_len, cfg.page_size
    ks = np.asarray(k_scale, np.float64)[:, None]
    vs = np.asarray(v_scale, np.float64)[:, None]
    for slot in range(pk.n_live):
        r = int(pk.slot_req[slot])
        for t in range(b):
            pos = int(pk.slot_pos0[slot]) + t
            page = int(page_table[r, pos // ps])
            k = k_new[slot * b + t]
            if rope_base > 0.0:
                k = rope_rotate(k, pos, rope_base)
            k_pool8[page, :, pos % ps, :] = e4m3_quantize(k, ks)
            v_pool8[page, :, pos % ps, :] = e4m3_quantize(v_new[slot * b + t], vs)


def wavefront_attn_fp8(cfg: Config, pk: Pack, q, k_pool8, v_pool8, k_scale,
                       v_scale, page_table, only_slots=None) -> np.ndarray:
    """wavefront_attn over 8-bit pages with the window resident in them: every
    key and value is what the page gives back, code * scale of its KV head, in
    float64; the queries are used as given."""
    ks = np.asarray(k_scale, np.float64)[None, :, None, None]
    vs = np.asarray(v_scale, np.float64)[None, :, None, None]
    kd = e4m3_decode(k_pool8) * ks
    vd = e4m3_decode(v_pool8) * vs
    return wavefront_attn(cfg, pk, q, None, None, kd, vd, page_table, only_slots)


def embed_gather(cfg: Config, pk: Pack, table):
    """Input embeddings of the packed window: row i of the result is the
    embedding-table row of the gathered token qtok[i] (Eq. 4 feeding the
    model's first layer), for the rows of live slots; rows of padding slots
    stay zero.  table [rows >= every token id in use, hidden]."""
    n = pk.n_live * cfg.block_len
    out = np.zeros((cfg.max_slots * cfg.block_len, table.shape[1]), table.dtype)
    for i in range(n):
        out[i] = table[int(pk.qtok[i])]
    return out


# --------------------------------------------------------------------------
# a3  top-1 prediction and its softmax confidence   (Sec. 2.1, before Eq. 1)
# --------------------------------------------------------------------------
def t2t_rows(cfg: Config, pk: Pack, logits):
    """x_hat_i = argmax_j z_ij and p_i = softmax(z_i)[x_hat_i] for live rows.

    logits [S*bl, V] float64.  READING: ties go to the lowest vocabulary
    index.  p = 1 / sum_j exp(z_j - max).  Padding rows: argmax -1, conf 0."""
    b = cfg.block_len
    n_rows = cfg.max_slots * b
    xhat = np.full(n_rows, -1, np.int32)
    conf = np.zeros(n_rows, np.float64)
    for i in range(pk.n_live * b):
        z = logits[i]
        m = z.max()
        xhat[i] = int(np.argmax(z))          # numpy returns first occurrence
        conf[i] = 1.0 / np.exp(z - m).sum()
    return xhat, conf


def lm_head_rows(cfg: Config, pk: Pack, x, w):
    """The row pass with the LM head in front of it: logits z = x W^T of the
    live rows (hidden states x [S*bl, hidden], head weights w [V, hidden], both
    float64), never rounded to a storage type, then exactly t2t_rows: top-1
    token (lowest index on ties) and its softmax confidence.  Sec. 3.1 notes
    that the readiness statistics come "from the current-step logits" at no
    extra cost; this is that pass taken straight from the head's output."""
    n = pk.n_live * cfg.block_len
    logits = np.zeros((cfg.max_slots * cfg.block_len, w.shape[0]), np.float64)
    logits[:n] = x[:n] @ w.T
    return t2t_rows(cfg, pk, logits)


# --------------------------------------------------------------------------
# a4 + a5  joint M2T u T2T update and per-block counts   (Eq. 1, Eq. 2)
# --------------------------------------------------------------------------
def t2t_update(cfg: Config, pk: Pack, st: State, xhat, conf):
    """Apply Eq. 1 to every live block, in place on st.tokens.

    Gamma = {x = [M] and p > tau_mask}  -> reveal (M2T).
    Delta = {x != x_hat and p > tau_edit and not prompt} -> overwrite (T2T).
    READING: Delta is taken on revealed positions only (the prose calls T2T an
    update of "an already revealed" position); identical to the literal set
    whenever tau_edit >= tau_mask.  Live blocks hold no prompt positions.
    Thresholds are binary32 values compared against the fp64 confidence.

    ``delta_literal = 1``: Delta exactly as Eq. 1 prints it, without the
    restriction to revealed positions: a masked position whose prediction is
    not [M] itself is updated as soon as p > tau_edit, whatever tau_mask says
    (it only matters when tau_edit < tau_mask).  Revealing a mask is M2T in
    the paper's terms whichever set it came through.

    ``force_progress = 1`` (READING; Eq. 1 is threshold-only and the paper
    names no fallback): if the oldest live block of a request went into the
    forward with masks and Eq. 1 revealed none of them, its masked position
    with the highest confidence (lowest position on ties; the plain fp64
    comparison of the confidences as given) is revealed (ACT_FORCED, counted
    as M2T).  Younger blocks are left to the thresholds:
    their context is still immature (Sec. 2.2).  The oldest block then loses a
    mask every step, so a request terminates whatever the logits do.

    Per slot: m0 = masks before the update, rdy = |{i in M_B: p_i >= tau_mask}|
    (numerator of Eq. 2; READING: M_B is the mask set that went into this
    forward), n_m2t, n_t2t, m1 = masks after, has_eos.
    Returns (action uint8 [S*bl], slot_stats int32 [S, 6])."""
    b = cfg.block_len
    tm = float(np.float32(cfg.tau_mask))
    te = float(np.float32(cfg.tau_edit))
    action = np.zeros(cfg.max_slots * b, np.uint8)
    stats = np.zeros((cfg.max_slots, 6), np.int32)
    for slot in range(pk.n_live):
        r, s = int(pk.slot_req[slot]), int(pk.slot_s[slot])
        g = int(st.L[r]) + s
        masked_before = []
        for t in range(b):
            i = slot * b + t
            col = g * b + t
            x = int(st.tokens[r, col])
            p = float(conf[i])
            if x == cfg.mask_id:
                masked_before.append(t)
                stats[slot, ST_M0] += 1
                if p >= tm:
                    stats[slot, ST_RDY] += 1
                in_gamma = p > tm
                in_delta = bool(cfg.delta_literal) and x != int(xhat[i]) and p > te
                if in_gamma or in_delta:
                    st.tokens[r, col] = xhat[i]
                    action[i] = ACT_M2T
                    stats[slot, ST_M2T] += 1
            elif x != int(xhat[i]) and p > te:
                st.tokens[r, col] = xhat[i]
                action[i] = ACT_T2T
                stats[slot, ST_T2T] += 1
        if (cfg.force_progress and s == 0 and masked_before
                and stats[slot, ST_M2T] == 0):
            best = masked_before[0]
            for t in masked_before[1:]:
                if conf[slot * b + t] > conf[slot * b + best]:
                    best = t
            st.tokens[r, g * b + best] = xhat[slot * b + best]
            action[slot * b + best] = ACT_FORCED
            stats[slot, ST_M2T] += 1
        for t in range(b):
            y = int(st.tokens[r, g * b + t])
            if y == cfg.mask_id:
                stats[slot, ST_M1] += 1
            if y == cfg.eos_id:
                stats[slot, ST_EOS] = 1
    return action, stats


# --------------------------------------------------------------------------
# a6 + a7  in-order retirement, KV freeze, gated admission   (Alg. 1 l.7-12)
# --------------------------------------------------------------------------
def readiness(m0: int, rdy: int) -> np.float32:
    """rho(B) of Eq. 2; rho = 1 when no masked position went into the forward.
    READING: evaluated in binary32 with a correctly rounded division."""
    if m0 == 0:
        return np.float32(1.0)
    return np.float32(rdy) / np.float32(m0)


def locally_finished(cfg: Config, m0, m1, n_upd, pe_new) -> bool:
    """Block-level commit signal (Sec. 2.1, last paragraph).  READING: once no
    masks remain the block gets up to S_pe further forwards and stops early on
    a forward that changes nothing; pe_new counts forwards that started with
    no masks, this one included."""
    return m1 == 0 and ((m0 == 0 and n_upd == 0) or pe_new >= cfg.s_pe)


def gate_commit(cfg: Config, pk: Pack, stats, st: State, k_win=None,
                v_win=None, k_pool=None, v_pool=None):
    """Retire, freeze KV, admit -- Alg. 1 lines 7-12 per request, in place.

    Retirement cascades over the maximal finished prefix of the window
    (the while of l.7) and stops after a block holding EOS (only a committed
    EOS terminates).  The retiring block's window K/V rows are copied to
    absolute positions [o_r, o_r + bl) of the request's pages (Eq. 6 for the
    committing block); frozen entries are never touched again.
    Admission (l.10, Eq. 3): READING at most one block per step, since a
    block admitted now has no current-step logits; the frontier is block R-1
    as it was in this forward, even if it has just retired; an empty window
    counts as rho = 1.  The new block is all [M].
    Returns (n_committed int32 [R], spawned uint8 [R], counters int32 [10])."""
    if cfg.batch_sync:
        return gate_commit_batch_sync(cfg, pk, stats, st, k_win, v_win,
                                      k_pool, v_pool)
    b, ps, W = cfg.block_len, cfg.page_size, cfg.wmax
    n_committed = np.zeros(cfg.max_requests, np.int32)
    spawned = np.zeros(cfg.max_requests, np.uint8)
    ctr = np.zeros(N_COUNTERS, np.int32)
    ctr[CT_LIVE_SLOTS] = pk.n_live
    theta = np.float32(cfg.theta_spawn)
    for r in range(cfg.max_requests):
        if st.active[r] != 1:
            continue
        first = int(pk.req_slot_begin[r])
        w = int(pk.req_slot_begin[r + 1]) - first
        assert w == int(st.R[r]) - int(st.L[r])
        pe_new, fin = [], []
        for s in range(w):
            m0, rdy, a, e, m1, _ = (int(v) for v in stats[first + s])
            pn = min(255, int(st.pe_done[r, s]) + (1 if m0 == 0 else 0))
            pe_new.append(pn)
            fin.append(locally_finished(cfg, m0, m1, a + e, pn))
            ctr[CT_M2T] += a
            ctr[CT_T2T] += e
        # retire in order
        c, eos = 0, False
        while c < w and fin[c]:
            if k_win is not None:
                P = int(st.prefix_len[r]) + c * b
                for t in range(b):
                    page = int(st.page_table[r, (P + t) // ps])
                    k_pool[page, :, (P + t) % ps, :] = k_win[(first + c) * b + t]
                    v_pool[page, :, (P + t) % ps, :] = v_win[(first + c) * b + t]
            c += 1
            if stats[first + c - 1, ST_EOS]:
                eos = True
                break
        st.L[r] += c
        st.prefix_len[r] += c * b
        for s in range(W):
            st.pe_done[r, s] = pe_new[s + c] if s + c < w else 0
        n_committed[r] = c
        ctr[CT_BLOCKS] += c
        ctr[CT_TOKENS] += c * b
        if eos or st.L[r] == cfg.max_blocks:
            st.active[r] = 2
            ctr[CT_FINISHED] += 1
            continue
        # gated admission
        if w > 0:
            rho = readiness(int(stats[first + w - 1, ST_M0]),
                            int(stats[first + w - 1, ST_RDY]))
        else:
            rho = np.float32(1.0)
        if (rho >= theta and st.R[r] - st.L[r] < W
                and st.R[r] < cfg.max_blocks):
            g = int(st.R[r])
            st.tokens[r, g * b:(g + 1) * b] = cfg.mask_id
            st.R[r] += 1
            st.pe_done[r, int(st.R[r] - st.L[r]) - 1] = 0
            spawned[r] = 1
            ctr[CT_SPAWNED] += 1
    ctr[CT_ACTIVE] = int((st.active == 1).sum())
    return n_committed, spawned, ctr


def gate_commit_batch_sync(cfg: Config, pk: Pack, stats, st: State,
                           k_win=None, v_win=None, k_pool=None, v_pool=None):
    """The batch-synchronous wavefront that Sec. 3.2 and the packing ablation
    (Sec. 4.5) set against per-sequence wavefronts: the same per-block
    predicates, but window position c retires only when it is finished in
    EVERY sequence still in the batch (``finished.all()``) and a block is
    admitted only when min_b rho_b clears theta_spawn.

    READING: the sequences keep their own (L_r, R_r) and move them together,
    which is the shared [L, R) whenever they start equal.  A sequence whose
    retired block holds EOS is done and leaves the reductions at once; the
    cascade goes on for the others.  The admission needs every remaining
    sequence to clear the gate and to have room (R - L < W, R < n): all of
    them get one new block or none does.  With one sequence this is
    gate_commit itself.  counters[CT_LOCKSTEP_COMMIT] = window positions
    retired by the batch this step, counters[CT_LOCKSTEP_ADMIT] = 1 if the
    batch admitted."""
    b, ps, W = cfg.block_len, cfg.page_size, cfg.wmax
    n_committed = np.zeros(cfg.max_requests, np.int32)
    spawned = np.zeros(cfg.max_requests, np.uint8)
    ctr = np.zeros(N_COUNTERS, np.int32)
    ctr[CT_LIVE_SLOTS] = pk.n_live
    theta = np.float32(cfg.theta_spawn)
    batch = [r for r in range(cfg.max_requests) if st.active[r] == 1]
    first, width, pe_new, fin = {}, {}, {}, {}
    for r in batch:
        first[r] = int(pk.req_slot_begin[r])
        width[r] = int(pk.req_slot_begin[r + 1]) - first[r]
        assert width[r] == int(st.R[r]) - int(st.L[r])
        pe_new[r], fin[r] = [], []
        for s in range(width[r]):
            m0, rdy, a, e, m1, _ = (int(v) for v in stats[first[r] + s])
            pn = min(255, int(st.pe_done[r, s]) + (1 if m0 == 0 else 0))
            pe_new[r].append(pn)
            fin[r].append(locally_finished(cfg, m0, m1, a + e, pn))
            ctr[CT_M2T] += a
            ctr[CT_T2T] += e
    # retire window position c in every sequence, or in none.  (A sequence
    # handed in with L == n already has nothing left: it is done at once, as
    # in gate_commit, and holds nobody back.)
    done = [r for r in batch if st.L[r] == cfg.max_blocks]
    alive = [r for r in batch if r not in done]
    c = 0
    while alive and all(c < width[r] and fin[r][c] for r in alive):
        for r in alive:
            if k_win is not None:
                P = int(st.prefix_len[r])
                for t in range(b):
                    page = int(st.page_table[r, (P + t) // ps])
                    k_pool[page, :, (P + t) % ps, :] = k_win[(first[r] + c) * b + t]
                    v_pool[page, :, (P + t) % ps, :] = v_win[(first[r] + c) * b + t]
            st.L[r] += 1
            st.prefix_len[r] += b
            n_committed[r] += 1
            if stats[first[r] + c, ST_EOS] or st.L[r] == cfg.max_blocks:
                done.append(r)
        alive = [r for r in alive if r not in done]
        c += 1
    ctr[CT_LOCKSTEP_COMMIT] = c
    for r in batch:
        k = int(n_committed[r])
        for s in range(W):
            st.pe_done[r, s] = pe_new[r][s + k] if s + k < width[r] else 0
        ctr[CT_BLOCKS] += k
        ctr[CT_TOKENS] += k * b
    for r in done:
        st.active[r] = 2
        ctr[CT_FINISHED] += 1
    # one admission decision for the batch
    left = [r for r in batch if r not in done]

    def clears(r):
        w = width[r]
        rho = (readiness(int(stats[first[r] + w - 1, ST_M0]),
                         int(stats[first[r] + w - 1, ST_RDY]))
               if w > 0 else np.float32(1.0))
        return bool(rho >= theta and st.R[r] - st.L[r] < W
                    and st.R[r] < cfg.max_blocks)

    if left and all(clears(r) for r in left):
        ctr[CT_LOCKSTEP_ADMIT] = 1
        for r in left:
            g = int(st.R[r])
            st.tokens[r, g * b:(g + 1) * b] = cfg.mask_id
            st.R[r] += 1
            st.pe_done[r, int(st.R[r] - st.L[r]) - 1] = 0
            spawned[r] = 1
            ctr[CT_SPAWNED] += 1
    ctr[CT_ACTIVE] = int((st.active == 1).sum())
    return n_committed, spawned, ctr


def decode_step(cfg: Config, st: State, logits, kv=None):
    """One step of Alg. 1 for the whole batch: pack, (attention is the model's
    business), Eq. 1 update of all live blocks, retire, admit.  ``logits`` is
    [S*bl, V] float64 in slot order for THIS step's packing."""
    pk = pack_wavefronts(cfg, st)
    xhat, conf = t2t_rows(cfg, pk, logits)
    action, stats = t2t_update(cfg, pk, st, xhat, conf)
    if kv is None:
        res = gate_commit(cfg, pk, stats, st)
    else:
        res = gate_commit(cfg, pk, stats, st, *kv)
    return pk, xhat, conf, action, stats, res


# --------------------------------------------------------------------------
# Independently written serial block-wise decoder (the W = 1 special case the
# paper calls "serial block-wise decoding", Sec. 2.2): one active block at a
# time, Eq. 1 until locally finished, then the next block.
# --------------------------------------------------------------------------
def serial_blockwise_decode(bl, n_blocks, vocab_mask_id, eos_id, tau_mask,
                            tau_edit, s_pe, logits_for, max_steps=10_000):
    """``logits_for(step, block)`` -> [bl, V] float64.  Returns (tokens
    [n_blocks*bl], list of (step, block) commit events, steps used)."""
    tm, te = float(np.float32(tau_mask)), float(np.float32(tau_edit))
    x = np.full(n_blocks * bl, vocab_mask_id, np.int64)
    events = []
    step = 0
    blk = 0
    post = 0
    while blk < n_blocks and step < max_steps:
        z = logits_for(step, blk)
        cur = x[blk * bl:(blk + 1) * bl]          # view
        had_mask = bool((cur == vocab_mask_id).any())
        if not had_mask:
            post += 1
        changed = 0
        for t in range(bl):
            e = np.exp(z[t] - z[t].max())
            p = float(e.max() / e.sum())
            top = int(np.flatnonzero(z[t] == z[t].max())[0])
            if cur[t] == vocab_mask_id:
                if p > tm:
                    cur[t] = top
                    changed += 1
            elif cur[t] != top and p > te:
                cur[t] = top
                changed += 1
        step += 1
        still = bool((cur == vocab_mask_id).any())
        done = (not still) and ((not had_mask and changed == 0) or post >= s_pe)
        if done:
            events.append((step - 1, blk))
            if (cur == eos_id).any():
                break
            blk += 1
            post = 0
    return x, events, step
