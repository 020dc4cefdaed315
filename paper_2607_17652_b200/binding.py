"""ctypes binding of libflowblock.so: argument marshalling only.

Every step of the hot path runs inside the CUDA library; this module turns
torch tensors into raw device pointers and calls the C entry points of the
same name.  There is no CPU fallback: if the library has not been built the
import of :func:`lib` raises.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libflowblock.so")

FB_OK = 0
FB_ERR_INVALID_ARG, FB_ERR_SHAPE, FB_ERR_ALIGNMENT = -1, -2, -3
FB_ERR_UNSUPPORTED, FB_ERR_WORKSPACE, FB_ERR_CUDA = -4, -5, -6
FB_ST_BAD_PAGE, FB_ST_BAD_TOKEN, FB_ST_BAD_STATE = 1, 2, 4
FB_ST_NAN_LOGIT, FB_ST_DEV_TIMEOUT = 8, 16
FB_ACT_NONE, FB_ACT_M2T, FB_ACT_T2T, FB_ACT_FORCED = 0, 1, 2, 3
FB_SLOT_STATS, FB_STEP_COUNTERS = 6, 10

EXPORTS = ["fb_create", "fb_destroy", "fb_last_error", "fb_workspace_bytes",
           "fb_pack_wavefronts", "fb_wavefront_attn", "fb_t2t_step",
           "fb_gate_commit", "fb_step_host", "fb_wavefront_attn_static",
           "fb_scatter_window_kv", "fb_embed_gather", "fb_lm_head_t2t",
           "fb_lm_head_workspace_bytes", "fb_set_tuning", "fb_attn_plan_host",
           "fb_scatter_window_kv_fp8", "fb_wavefront_attn_fp8"]


class fb_config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in (
        "max_requests", "wmax", "block_len", "n_q_heads", "n_kv_heads",
        "head_dim", "page_size", "num_pages", "max_pages_per_req", "vocab",
        "mask_id", "eos_id", "max_blocks", "s_pe")] + \
        [(n, C.c_float) for n in ("tau_mask", "tau_edit", "theta_spawn",
                                  "sm_scale")] + \
        [("window_in_pages", C.c_int32), ("batch_sync", C.c_int32),
         ("delta_literal", C.c_int32), ("force_progress", C.c_int32),
         ("kv_fp8", C.c_int32)]


class fb_tuning(C.Structure):
    _fields_ = [("attn_target_items", C.c_int32),
                ("attn_min_chunk_tiles", C.c_int32),
                ("attn_pair", C.c_int32), ("reserved", C.c_int32),
                ("wait_cycles", C.c_int64)]


class fb_state(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in (
        "active", "prefix_len", "L", "R", "tokens", "pe_done", "page_table")]


class fb_pack(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in (
        "n_live", "slot_req", "slot_s", "slot_pos0", "slot_kv_len",
        "slot_flags", "req_slot_begin", "qtok", "pos")]


class fb_host_io(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in (
        "h_q", "h_k_win", "h_v_win", "h_logits", "h_n_committed", "h_spawned",
        "h_step_counters", "h_status")] + [("n_rows", C.c_int64)]


class fb_device_bufs(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in (
        "q", "k_win", "v_win", "out", "logits", "k_pool", "v_pool", "argmax",
        "conf", "action", "slot_stats", "n_committed", "spawned",
        "step_counters", "status", "ws")]


_lib = None


def lib() -> C.CDLL:
    """The loaded CUDA library.  Raises if it is missing (no fallback)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with "
                "`python -m paper_2607_17652_b200.build`; there is no CPU "
                "fallback for the FlowBlock hot path")
        l = C.CDLL(LIB_PATH)
        P, I = C.c_void_p, C.c_int
        l.fb_create.argtypes = [C.POINTER(fb_config), C.POINTER(P)]
        l.fb_destroy.argtypes = [P]
        l.fb_last_error.argtypes = [P]
        l.fb_last_error.restype = C.c_char_p
        l.fb_workspace_bytes.argtypes = [P]
        l.fb_workspace_bytes.restype = C.c_size_t
        l.fb_set_tuning.argtypes = [P, C.POINTER(fb_tuning)]
        l.fb_attn_plan_host.argtypes = [P, P, P, C.c_int32, P]
        l.fb_pack_wavefronts.argtypes = [P, C.POINTER(fb_state),
                                         C.POINTER(fb_pack), P, P, P]
        l.fb_wavefront_attn.argtypes = [P, C.POINTER(fb_pack)] + [P] * 10
        l.fb_t2t_step.argtypes = [P, C.POINTER(fb_pack), P,
                                  C.POINTER(fb_state)] + [P] * 6
        l.fb_gate_commit.argtypes = [P, C.POINTER(fb_pack), P,
                                     C.POINTER(fb_state)] + [P] * 9
        l.fb_wavefront_attn_static.argtypes = [P, C.POINTER(fb_state),
                                               C.POINTER(fb_pack)] + [P] * 8
        l.fb_scatter_window_kv.argtypes = [P, C.POINTER(fb_pack)] + [P] * 5 + \
            [C.c_float, P, P]
        l.fb_scatter_window_kv_fp8.argtypes = [P, C.POINTER(fb_pack)] + [P] * 7 + \
            [C.c_float, P, P]
        l.fb_wavefront_attn_fp8.argtypes = [P, C.POINTER(fb_pack)] + [P] * 10
        l.fb_embed_gather.argtypes = [P, C.POINTER(fb_pack), P, C.c_int32,
                                      C.c_int32, P, P, P]
        l.fb_lm_head_workspace_bytes.argtypes = [P]
        l.fb_lm_head_workspace_bytes.restype = C.c_size_t
        l.fb_lm_head_t2t.argtypes = [P, C.POINTER(fb_pack), P, P, C.c_int32,
                                     C.POINTER(fb_state)] + [P] * 7
        l.fb_step_host.argtypes = [P, C.POINTER(fb_state), C.POINTER(fb_pack),
                                   C.POINTER(fb_device_bufs),
                                   C.POINTER(fb_host_io), P]
        for n in EXPORTS:
            if n not in ("fb_last_error", "fb_workspace_bytes",
                         "fb_lm_head_workspace_bytes"):
                getattr(l, n).restype = I
        _lib = l
    return _lib


class FlowBlockError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__(f"flowblock error {code}: {msg}")
        self.code = code


def _ptr(t) -> int | None:
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


class Context:
    """Owns one fb_ctx.  ``tuning``: optional dict of fb_tuning fields."""

    def __init__(self, tuning=None, **cfg):
        self.cfg = fb_config(**cfg)
        self._h = C.c_void_p()
        rc = lib().fb_create(C.byref(self.cfg), C.byref(self._h))
        if rc != FB_OK:
            raise FlowBlockError(rc, lib().fb_last_error(None).decode())
        if tuning:
            self.set_tuning(**tuning)

    def set_tuning(self, **tuning):
        """fb_set_tuning; buffers sized by workspace_bytes() must be allocated after it."""
        t = fb_tuning(**tuning)
        self.check(lib().fb_set_tuning(self._h, C.byref(t)))

    def attn_plan(self, prefix_len, live_blocks) -> dict:
        """fb_attn_plan_host: what the attention work list of such a batch holds."""
        p = np.ascontiguousarray(prefix_len, np.int32)
        w = np.ascontiguousarray(live_blocks, np.int32)
        out = np.zeros(12, np.int32)
        self.check(lib().fb_attn_plan_host(self._h, p.ctypes.data, w.ctypes.data, len(p), out.ctypes.data))
        names = ("units", "items", "parts", "max_units", "max_items", "max_parts")
        d = dict(zip(names, map(int, out[:6])))                      # the one-CTA kernel's list
        d["pair"] = dict(zip(names, map(int, out[6:])))              # the CTA-pair kernel's list
        return d

    def __del__(self):
        try:
            if self._h:
                lib().fb_destroy(self._h)
                self._h = C.c_void_p()
        except Exception:
            pass

    @property
    def handle(self):
        return self._h

    @property
    def max_slots(self):
        return self.cfg.max_requests * self.cfg.wmax

    def workspace_bytes(self) -> int:
        return lib().fb_workspace_bytes(self._h)

    def check(self, rc):
        if rc != FB_OK:
            raise FlowBlockError(rc, lib().fb_last_error(self._h).decode())


@dataclass
class DeviceState:
    active: torch.Tensor
    prefix_len: torch.Tensor
    L: torch.Tensor
    R: torch.Tensor
    tokens: torch.Tensor
    pe_done: torch.Tensor
    page_table: torch.Tensor

    @classmethod
    def from_numpy(cls, device, active, prefix_len, L, R, tokens, pe_done,
                   page_table):
        f = lambda a, dt: torch.from_numpy(np.ascontiguousarray(a)).to(dt).to(device)
        return cls(f(active, torch.int32), f(prefix_len, torch.int32),
                   f(L, torch.int32), f(R, torch.int32),
                   f(tokens, torch.int32), f(pe_done, torch.uint8),
                   f(page_table, torch.int32))

    def c(self) -> fb_state:
        return fb_state(*(_ptr(getattr(self, n)) for n, _ in fb_state._fields_))

    def to_numpy(self):
        return {n: getattr(self, n).cpu().numpy() for n, _ in fb_state._fields_}


@dataclass
class PackBuffers:
    n_live: torch.Tensor
    slot_req: torch.Tensor
    slot_s: torch.Tensor
    slot_pos0: torch.Tensor
    slot_kv_len: torch.Tensor
    slot_flags: torch.Tensor
    req_slot_begin: torch.Tensor
    qtok: torch.Tensor
    pos: torch.Tensor

    @classmethod
    def alloc(cls, ctx: Context, device):
        S, b, R = ctx.max_slots, ctx.cfg.block_len, ctx.cfg.max_requests
        z = lambda n: torch.full((n,), -7, dtype=torch.int32, device=device)
        return cls(z(1), z(S), z(S), z(S), z(S), z(S), z(R + 1), z(S * b),
                   z(S * b))

    def c(self) -> fb_pack:
        return fb_pack(*(_ptr(getattr(self, n)) for n, _ in fb_pack._fields_))

    def to_numpy(self):
        return {n: getattr(self, n).cpu().numpy() for n, _ in fb_pack._fields_}


def alloc_workspace(ctx: Context, device) -> torch.Tensor:
    n = ctx.workspace_bytes()
    return torch.zeros((n + 255) // 256 * 256, dtype=torch.uint8, device=device)


# ----------------------------------------------------------------- the calls
def fb_pack_wavefronts(ctx: Context, st: DeviceState, pk: PackBuffers, ws,
                       status, stream=None):
    s, p = st.c(), pk.c()
    ctx.check(lib().fb_pack_wavefronts(ctx.handle, C.byref(s), C.byref(p),
                                       _ptr(ws), _ptr(status), _stream(stream)))


def fb_wavefront_attn(ctx: Context, pk: PackBuffers, q, k_win, v_win, k_pool,
                      v_pool, page_table, out, ws, status, stream=None):
    p = pk.c()
    ctx.check(lib().fb_wavefront_attn(
        ctx.handle, C.byref(p), _ptr(q), _ptr(k_win), _ptr(v_win),
        _ptr(k_pool), _ptr(v_pool), _ptr(page_table), _ptr(out), _ptr(ws),
        _ptr(status), _stream(stream)))


def fb_scatter_window_kv(ctx: Context, pk: PackBuffers, page_table, k_new, v_new,
                         k_pool, v_pool, status, rope_base: float = 0.0,
                         stream=None):
    """Eq. 6 as data movement (contexts with window_in_pages=1)."""
    p = pk.c()
    ctx.check(lib().fb_scatter_window_kv(
        ctx.handle, C.byref(p), _ptr(page_table), _ptr(k_new), _ptr(v_new),
        _ptr(k_pool), _ptr(v_pool), C.c_float(rope_base), _ptr(status),
        _stream(stream)))


def fb_scatter_window_kv_fp8(ctx: Context, pk: PackBuffers, page_table, k_new, v_new,
                             k_pool8, v_pool8, k_scale, v_scale, status,
                             rope_base: float = 0.0, stream=None):
    """Eq. 6 into 8-bit (E4M3) pages with per-KV-head scales."""
    p = pk.c()
    ctx.check(lib().fb_scatter_window_kv_fp8(
        ctx.handle, C.byref(p), _ptr(page_table), _ptr(k_new), _ptr(v_new),
        _ptr(k_pool8), _ptr(v_pool8), _ptr(k_scale), _ptr(v_scale),
        C.c_float(rope_base), _ptr(status), _stream(stream)))


def fb_wavefront_attn_fp8(ctx: Context, pk: PackBuffers, q, k_pool8, v_pool8,
                          k_scale, v_scale, page_table, out, ws, status,
                          stream=None):
    """Attention over 8-bit (E4M3) pages, window resident in the pages."""
    p = pk.c()
    ctx.check(lib().fb_wavefront_attn_fp8(
        ctx.handle, C.byref(p), _ptr(q), _ptr(k_pool8), _ptr(v_pool8),
        _ptr(k_scale), _ptr(v_scale), _ptr(page_table), _ptr(out), _ptr(ws),
        _ptr(status), _stream(stream)))


def fb_embed_gather(ctx: Context, pk: PackBuffers, table, x, status, stream=None):
    """x[i] = table[qtok[i]] for the rows of live slots (Eq. 4 feeding the model)."""
    p = pk.c()
    ctx.check(lib().fb_embed_gather(
        ctx.handle, C.byref(p), _ptr(table), int(table.shape[0]),
        int(table.shape[1]), _ptr(x), _ptr(status), _stream(stream)))


def fb_wavefront_attn_static(ctx: Context, st: DeviceState, pk: PackBuffers, q,
                             k_win, v_win, k_pool, v_pool, out, status,
                             stream=None):
    """Attention for callers that cannot allocate: no workspace argument, the
    scratch is an array inside the library (see the header for its limits)."""
    s, p = st.c(), pk.c()
    ctx.check(lib().fb_wavefront_attn_static(
        ctx.handle, C.byref(s), C.byref(p), _ptr(q), _ptr(k_win), _ptr(v_win),
        _ptr(k_pool), _ptr(v_pool), _ptr(out), _ptr(status), _stream(stream)))


def fb_t2t_step(ctx: Context, pk: PackBuffers, logits, st: DeviceState, argmax,
                conf, action, slot_stats, status, stream=None):
    s, p = st.c(), pk.c()
    ctx.check(lib().fb_t2t_step(
        ctx.handle, C.byref(p), _ptr(logits), C.byref(s), _ptr(argmax),
        _ptr(conf), _ptr(action), _ptr(slot_stats), _ptr(status),
        _stream(stream)))


def fb_lm_head_t2t(ctx: Context, pk: PackBuffers, x, w, st: DeviceState, argmax,
                   conf, action, slot_stats, ws, status, stream=None):
    """fb_t2t_step with the LM head fused in front (logits never written)."""
    s, p = st.c(), pk.c()
    ctx.check(lib().fb_lm_head_t2t(
        ctx.handle, C.byref(p), _ptr(x), _ptr(w), int(x.shape[1]), C.byref(s),
        _ptr(argmax), _ptr(conf), _ptr(action), _ptr(slot_stats), _ptr(ws),
        _ptr(status), _stream(stream)))


def fb_gate_commit(ctx: Context, pk: PackBuffers, slot_stats, st: DeviceState,
                   k_win, v_win, k_pool, v_pool, n_committed, spawned,
                   step_counters, status, stream=None):
    s, p = st.c(), pk.c()
    ctx.check(lib().fb_gate_commit(
        ctx.handle, C.byref(p), _ptr(slot_stats), C.byref(s), _ptr(k_win),
        _ptr(v_win), _ptr(k_pool), _ptr(v_pool), _ptr(n_committed),
        _ptr(spawned), _ptr(step_counters), _ptr(status), _stream(stream)))


def fb_step_host(ctx: Context, st: DeviceState, pk: PackBuffers, dev: dict,
                 host: dict, stream=None):
    """dev / host: dicts of tensors keyed by the C field names."""
    s, p = st.c(), pk.c()
    d = fb_device_bufs(*(_ptr(dev[n]) for n, _ in fb_device_bufs._fields_))
    h = fb_host_io(*(_ptr(host[n]) for n, _ in fb_host_io._fields_[:-1]),
                   int(host.get("n_rows", 0)))
    ctx.check(lib().fb_step_host(ctx.handle, C.byref(s), C.byref(p),
                                 C.byref(d), C.byref(h), _stream(stream)))


class StepBuffers:
    """Device outputs of one step, allocated once (fixed shapes)."""

    def __init__(self, ctx: Context, device):
        S, b, R = ctx.max_slots, ctx.cfg.block_len, ctx.cfg.max_requests
        c = ctx.cfg
        self.out = torch.zeros(S * b, c.n_q_heads, c.head_dim,
                               dtype=torch.bfloat16, device=device)
        self.argmax = torch.full((S * b,), -9, dtype=torch.int32, device=device)
        self.conf = torch.full((S * b,), -1.0, dtype=torch.float32, device=device)
        self.action = torch.full((S * b,), 9, dtype=torch.uint8, device=device)
        self.slot_stats = torch.full((S, FB_SLOT_STATS), -9, dtype=torch.int32,
                                     device=device)
        self.n_committed = torch.full((R,), -9, dtype=torch.int32, device=device)
        self.spawned = torch.full((R,), 9, dtype=torch.uint8, device=device)
        self.step_counters = torch.full((FB_STEP_COUNTERS,), -9,
                                        dtype=torch.int32, device=device)
        self.status = torch.zeros(1, dtype=torch.int32, device=device)
        self.ws = alloc_workspace(ctx, device)
