#!/usr/bin/env python
"""Benchmark of the packed-wavefront decode step on B200.

A step = fb_pack_wavefronts -> fb_wavefront_attn -> fb_t2t_step ->
fb_gate_commit over one batch of seeded synthetic input.  Prints ONE JSON line
(rank 0).  `--impl reference` times the fp64 CPU oracle on a bounded sample
of the same workload instead.

Units
  value      whole-step throughput: algorithmic attention FLOPs of one step
             (4 d sum_live-slots bl Hq kv_len) / device time of the whole step,
             in TFLOP/s, inputs resident in HBM
  kernels    per-call device times inside the same timed steps, with the two
             figures the metric names: attention TFLOP/s and T2T-step GB/s
  e2e        the same step through fb_step_host: pinned host q / k_win / v_win
             / logits copied in, decisions copied out, inside the timed region
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "packed-wavefront attn TFLOP/s & T2T-step GB/s (fraction of B200 peak)"
DEFAULT_WORKLOAD = 2
KERNELS_PER_STEP = 6   # pack, attention, split-KV combine, T2T rows, T2T update, gate/commit
# dram__bytes_read.sum + dram__bytes_write.sum from the ncu captures summarised
# under profiles/, as a ratio to the algorithmic bytes of the captured (smaller)
# case of the same workload; a full launch's traffic is that ratio times its
# algorithmic bytes (traffic grows in proportion to the requests processed).
NCU_TRAFFIC_RATIO = {("attn", 2): (1397.7 + 33.5) / 1366.9,   # profiles/wavefront_attn_cfg2_dram.txt (full size)
                     ("t2t", 2): (504.38 + 4.62) / 504.4}      # profiles/t2t_rows_cfg2_16req.txt


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return dict(hbm_gbs=d["hbm_gbs"], bf16_tflops=d["bf16_tflops"],
                    bf16_tflops_sustained=d.get("bf16_tflops_sustained"),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0,
                source="fallback")


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while timing."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_id: str):
        self.gpu_id, self.proc, self.lines = gpu_id, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", self.gpu_id, f"--query-gpu={self.Q}",
                 "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0, t1):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ts, line in self.lines:
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                c, m = float(f[0]), float(f[1])
            except ValueError:
                continue
            mx = m
            if t0 - 0.05 <= ts <= t1 + 0.15:
                sm.append(c)
                for n, v in zip(names, f[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": mx,
                "samples": len(sm), "reasons": sorted(reasons)}


def attn_flops(stc) -> float:
    wl = stc.wl
    tot = 0
    for r in range(wl.n_requests):
        if stc.active[r] != 1:
            continue
        for s in range(int(stc.R[r] - stc.L[r])):
            tot += wl.block_len * wl.n_q_heads * (int(stc.prefix_len[r]) + (s + 1) * wl.block_len)
    return 4.0 * wl.head_dim * tot


def attn_bytes(stc) -> float:
    """K/V read once per request and KV head + Q read + O written."""
    wl = stc.wl
    kv = 0
    rows = 0
    for r in range(wl.n_requests):
        if stc.active[r] != 1:
            continue
        w = int(stc.R[r] - stc.L[r])
        kv += int(stc.prefix_len[r]) + w * wl.block_len
        rows += w * wl.block_len
    return 2.0 * (2 * kv * wl.n_kv_heads * wl.head_dim + 2 * rows * wl.n_q_heads * wl.head_dim)


def t2t_bytes(stc, n_live) -> float:
    wl = stc.wl
    rows = n_live * wl.block_len
    return rows * (2.0 * wl.vocab + 4 + 4 + 1 + 4) + n_live * 24


def pick_workload(args):
    import dataclasses
    from paper_2607_17652_b200 import synth
    wl = synth.WORKLOADS[args.workload]
    if args.requests:
        wl = dataclasses.replace(wl, n_requests=args.requests, name=f"{wl.name}[{args.requests} requests]")
    return wl


def build_inputs(wl, seed):
    from paper_2607_17652_b200 import synth
    stc = synth.make_structure(wl, seed)
    tokens = synth.make_tokens(stc)
    n_live = synth.n_live_slots(stc)
    z, tokens = synth.make_logits(stc, tokens, n_rows=n_live * wl.block_len)
    attn = synth.make_attn_inputs(stc)
    return stc, tokens, n_live, z, attn


def combine_ranks(times_ms, work, device, world):
    """Whole-job figures from per-rank ones: every rank ran its own batch
    (replicas, no data-path collective), so times combine as the MAX over
    ranks and work as the SUM."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(times_ms, dtype=torch.float64, device=device)
    w = torch.tensor(work, dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(w, op=dist.ReduceOp.SUM)
    return [float(x) for x in t.cpu()], [float(x) for x in w.cpu()]


def free_port() -> int:
    import socket
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def launch_replicas(args) -> int:
    """`--gpus N` with N > 1 and no launcher environment: start the N ranks
    ourselves (one process per GPU, the same command line under
    torch.distributed.run on 127.0.0.1) and return their exit code."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def replica_env(args):
    """(rank, world, local rank) of this process.  Under a launcher the world
    is what was launched; a --gpus that disagrees with it is reported."""
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus and rank == 0:
        print(f"bench.py: --gpus {args.gpus} but {world} rank(s) were launched; reporting n_gpus = {world}",
              file=sys.stderr)
    return rank, world, local


def gather_ranks(record: dict, world):
    """One small record per rank, collected on every rank (host objects: no
    device memory is exchanged)."""
    import torch.distributed as dist
    if world == 1:
        return [record]
    out = [None] * world
    dist.all_gather_object(out, record)
    return out


def run_dry(args):
    """`--dry-run-cpu`: the replica plumbing without a GPU -- ranks over gloo,
    rank-dependent seeds, the MAX-of-times / SUM-of-work reduction and the JSON
    line -- with placeholder times and no kernel.  For tests of the launcher."""
    import torch.distributed as dist
    from paper_2607_17652_b200 import synth
    rank, world, local = replica_env(args)
    if world > 1:
        dist.init_process_group("gloo")
    wl = synth.tiny_workload()
    stc = synth.make_structure(wl, synth.BASE_SEED + wl.index + 1000 * rank)
    flops = attn_flops(stc)
    (ms, e2e_ms), (flops_all,) = combine_ranks([1.0 + rank, 10.0 + rank], [flops], "cpu", world)
    ranks = gather_ranks({"rank": rank, "local_rank": local, "seed": stc.seed, "attn_flops": flops}, world)
    if rank == 0:
        print(json.dumps({"metric": METRIC, "dry_run": True, "value": flops_all / ms / 1e9, "n_gpus": world,
                          "ms_per_step": ms, "scaling": "weak",
                          "config": {"workload": wl.name, "parallelism": f"replicas x{world}"},
                          "e2e": {"ms_per_step": e2e_ms}, "ranks": ranks}), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_fp8_only(args):
    """`--only attn_fp8`: fb_wavefront_attn_fp8 alone on the workload's structure (8-bit pools of
    N(0,1) values quantised on the device, window scattered once), for profiler captures."""
    import torch
    from paper_2607_17652_b200 import binding as B, synth
    dev = "cuda:0"
    torch.cuda.set_device(0)
    wl = pick_workload(args)
    stc = synth.make_structure(wl, synth.BASE_SEED + wl.index)
    tokens = synth.make_tokens(stc)
    ctx = B.Context(kv_fp8=1, **synth.config_dict(stc, window_in_pages=1))
    st = B.DeviceState.from_numpy(dev, stc.active, stc.prefix_len, stc.L, stc.R, tokens,
                                  np.zeros((wl.n_requests, wl.wmax), np.uint8), stc.page_table)
    pk = B.PackBuffers.alloc(ctx, dev)
    sb = B.StepBuffers(ctx, dev)
    gen = torch.Generator(device=dev); gen.manual_seed(stc.seed)
    rows = ctx.max_slots * wl.block_len
    q = torch.randn(rows, wl.n_q_heads, wl.head_dim, device=dev, generator=gen).to(torch.bfloat16)
    kw = torch.randn(rows, wl.n_kv_heads, wl.head_dim, device=dev, generator=gen).to(torch.bfloat16)
    vw = torch.randn(rows, wl.n_kv_heads, wl.head_dim, device=dev, generator=gen).to(torch.bfloat16)
    ks = torch.full((wl.n_kv_heads,), 6.0 / 448.0, device=dev)
    vs = ks.clone()
    shape = (stc.num_pages, wl.n_kv_heads, wl.page_size, wl.head_dim)
    pools = []
    for _ in range(2):
        pool = torch.empty(shape, dtype=torch.uint8, device=dev)
        for p0 in range(0, shape[0], 2048):
            x = torch.randn(pool[p0:p0 + 2048].shape, device=dev, generator=gen) / ks[None, :, None, None]
            pool[p0:p0 + 2048] = x.clamp_(-448.0, 448.0).to(torch.float8_e4m3fn).view(torch.uint8)
        pools.append(pool)
    k8, v8 = pools
    B.fb_pack_wavefronts(ctx, st, pk, sb.ws, sb.status)
    B.fb_scatter_window_kv_fp8(ctx, pk, st.page_table, kw, vw, k8, v8, ks, vs, sb.status)
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    for i in range(args.warmup + args.steps):
        e = ev[i - args.warmup] if i >= args.warmup else None
        if e: e[0].record()
        B.fb_wavefront_attn_fp8(ctx, pk, q, k8, v8, ks, vs, st.page_table, sb.out, sb.ws, sb.status)
        if e: e[1].record()
    torch.cuda.synchronize()
    ms = float(np.mean([a.elapsed_time(b) for a, b in ev]))
    peaks = load_peaks()
    tf = attn_flops(stc) / ms / 1e9
    print(json.dumps({"metric": METRIC, "only": "attn_fp8", "config": {"workload": wl.name, "requests": wl.n_requests},
                      "kernels": {"attn_ms": round(ms, 4), "attn_tflops": round(tf, 2)},
                      "frac_of_fp8_peak": round(tf / (2.0 * peaks["bf16_tflops"]), 4),
                      "device_status": int(sb.status.item())}), flush=True)


# ---------------------------------------------------------------- our arm
def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2607_17652_b200 import binding as B, synth

    rank, world, local = replica_env(args)
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    if world > 1:
        # replicas: NCCL only carries the MAX-of-times / SUM-of-work reduction at the end
        dist.init_process_group("nccl", device_id=torch.device(dev))
    wl = pick_workload(args)
    seed = synth.BASE_SEED + wl.index + 1000 * rank     # each rank its own batch
    stc, tokens, n_live, z_live, attn = build_inputs(wl, seed)
    stc_init = stc
    tuning = dict(attn_pair=int(args.pair), attn_target_items=args.target_items, attn_min_chunk_tiles=args.min_chunk)
    ctx = B.Context(tuning=tuning if any(tuning.values()) else None, **synth.config_dict(stc))
    st = B.DeviceState.from_numpy(dev, stc.active, stc.prefix_len, stc.L, stc.R, tokens,
                                  np.zeros((wl.n_requests, wl.wmax), np.uint8), stc.page_table)
    pk = B.PackBuffers.alloc(ctx, dev)
    sb = B.StepBuffers(ctx, dev)
    rows = ctx.max_slots * wl.block_len
    logits = torch.zeros(rows, wl.vocab, dtype=torch.bfloat16, device=dev)
    logits[:z_live.shape[0]].copy_(z_live)
    q, kw, vw, kp, vp = (t.to(dev) for t in attn)
    stream = torch.cuda.current_stream()

    only = args.only

    def step(ev=None):
        if ev: ev[0].record(stream)
        if only == "all" or ev is None:
            B.fb_pack_wavefronts(ctx, st, pk, sb.ws, sb.status, stream)
        if ev: ev[1].record(stream)
        if only in ("all", "attn"):
            B.fb_wavefront_attn(ctx, pk, q, kw, vw, kp, vp, st.page_table, sb.out, sb.ws, sb.status, stream)
        if ev: ev[2].record(stream)
        if only in ("all", "t2t"):
            B.fb_t2t_step(ctx, pk, logits, st, sb.argmax, sb.conf, sb.action, sb.slot_stats, sb.status, stream)
        if ev: ev[3].record(stream)
        if only == "all":
            B.fb_gate_commit(ctx, pk, sb.slot_stats, st, kw, vw, kp, vp, sb.n_committed, sb.spawned,
                             sb.step_counters, sb.status, stream)
        if ev: ev[4].record(stream)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def device_structure():
        """The workload structure as it stands on the device (commits and
        admissions of earlier steps move L, R and the prefix lengths)."""
        import dataclasses
        g = st.to_numpy()
        cur = dataclasses.replace(stc)
        cur.active, cur.prefix_len, cur.L, cur.R = g["active"], g["prefix_len"], g["L"], g["R"]
        return cur

    for _ in range(args.warmup):
        step()
    barrier()
    stc0 = device_structure()
    uuid = str(torch.cuda.get_device_properties(local).uuid)
    sampler = ClockSampler(uuid if uuid.startswith("GPU-") else "GPU-" + uuid)
    sampler.start()
    time.sleep(0.2)
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(args.steps)]
    barrier()
    t0 = time.time()
    # Workloads whose inputs fit in the 126 MB L2 (cfg0, cfg1) would otherwise be timed warm: a 256 MB write
    # between the timed steps evicts them; the step time is then the sum of the steps, not the span.
    in_bytes = sum(t.numel() * t.element_size() for t in (q, kw, vw, kp, vp)) + n_live * wl.block_len * wl.vocab * 2
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if in_bytes < (200 << 20) else None
    for k in range(args.steps):
        if flush is not None:
            flush.fill_(k & 0xFF)
        step(evs[k])
    barrier()
    t1 = time.time()
    seg = np.array([[e[i].elapsed_time(e[i + 1]) for i in range(4)] for e in evs])  # ms
    per_step = np.array([e[0].elapsed_time(e[4]) for e in evs])
    total_ms = evs[0][0].elapsed_time(evs[-1][4]) if flush is None else float(per_step.sum())
    status = int(sb.status.item())
    counters = sb.step_counters.cpu().numpy().tolist()
    stc1 = device_structure()

    # ---------------------- next row: Eq. 6 as data movement (window in pages)
    nxt = None
    if only == "all" and world == 1:
        ctx2 = B.Context(**synth.config_dict(stc, window_in_pages=1))
        pk2 = B.PackBuffers.alloc(ctx2, dev)
        ws2 = B.alloc_workspace(ctx2, dev)
        n2 = max(3, min(args.steps, 10))
        ev2 = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(n2)]
        for k in range(3 + n2):
            B.fb_pack_wavefronts(ctx2, st, pk2, ws2, sb.status, stream)
            e = ev2[k - 3] if k >= 3 else None
            if e: e[0].record(stream)
            B.fb_scatter_window_kv(ctx2, pk2, st.page_table, kw, vw, kp, vp, sb.status, 10000.0, stream)
            if e: e[1].record(stream)
            B.fb_wavefront_attn(ctx2, pk2, q, None, None, kp, vp, st.page_table, sb.out, ws2, sb.status, stream)
            if e: e[2].record(stream)
        barrier()
        sc_ms = float(np.mean([e[0].elapsed_time(e[1]) for e in ev2]))
        ra_ms = float(np.mean([e[1].elapsed_time(e[2]) for e in ev2]))
        live_now = synth.n_live_slots(device_structure())
        sc_bytes = 2.0 * 2 * live_now * wl.block_len * wl.n_kv_heads * wl.head_dim * 2      # K and V, read + write
        nxt = {"scatter_window_kv": {"ms": round(sc_ms, 4), "bytes": sc_bytes, "rope": True,
                                     "gbs": round(sc_bytes / sc_ms / 1e6, 1)},
               "attn_window_in_pages": {"ms": round(ra_ms, 4),
                                        "tflops": round(attn_flops(device_structure()) / ra_ms / 1e9, 2)}}
        if wl.head_dim == 128:
            # next row: the KV pages in 8 bits (FP8 E4M3, per-KV-head scales): scatter = quantiser, attention
            # with both products as 8-bit MMAs.  Pools of N(0,1) values quantised on the device.
            gen8 = torch.Generator(device=dev); gen8.manual_seed(seed + 78)
            ks8 = torch.full((wl.n_kv_heads,), 6.0 / 448.0, device=dev) * (0.5 + 1.5 * torch.rand(wl.n_kv_heads, device=dev, generator=gen8))
            vs8 = torch.full((wl.n_kv_heads,), 6.0 / 448.0, device=dev) * (0.5 + 1.5 * torch.rand(wl.n_kv_heads, device=dev, generator=gen8))
            kp8 = torch.empty(kp.shape, dtype=torch.uint8, device=dev)
            vp8 = torch.empty(vp.shape, dtype=torch.uint8, device=dev)
            for pool, sc in ((kp8, ks8), (vp8, vs8)):
                for p0 in range(0, pool.shape[0], 2048):
                    x = torch.randn(pool[p0:p0 + 2048].shape, device=dev, generator=gen8) / sc[None, :, None, None]
                    pool[p0:p0 + 2048] = x.clamp_(-448.0, 448.0).to(torch.float8_e4m3fn).view(torch.uint8)
            ctx8 = B.Context(kv_fp8=1, **synth.config_dict(stc, window_in_pages=1))
            pk8 = B.PackBuffers.alloc(ctx8, dev)
            ws8 = B.alloc_workspace(ctx8, dev)
            ev8 = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(n2)]
            for k in range(3 + n2):
                B.fb_pack_wavefronts(ctx8, st, pk8, ws8, sb.status, stream)
                e = ev8[k - 3] if k >= 3 else None
                if e: e[0].record(stream)
                B.fb_scatter_window_kv_fp8(ctx8, pk8, st.page_table, kw, vw, kp8, vp8, ks8, vs8, sb.status, 10000.0, stream)
                if e: e[1].record(stream)
                B.fb_wavefront_attn_fp8(ctx8, pk8, q, kp8, vp8, ks8, vs8, st.page_table, sb.out, ws8, sb.status, stream)
                if e: e[2].record(stream)
            barrier()
            s8_ms = float(np.mean([e[0].elapsed_time(e[1]) for e in ev8]))
            a8_ms = float(np.mean([e[1].elapsed_time(e[2]) for e in ev8]))
            cur = device_structure()
            kv_tokens = sum(int(cur.prefix_len[r]) + int(cur.R[r] - cur.L[r]) * wl.block_len
                            for r in range(wl.n_requests) if cur.active[r] == 1)
            a8_bytes = 2.0 * kv_tokens * wl.n_kv_heads * wl.head_dim + 2.0 * 2 * live_now * wl.block_len * wl.n_q_heads * wl.head_dim
            nxt["attn_fp8_pages"] = {"ms": round(a8_ms, 4), "tflops": round(attn_flops(cur) / a8_ms / 1e9, 2),
                                     "algorithmic_bytes": a8_bytes, "scatter_quantise_ms": round(s8_ms, 4),
                                     "speedup_vs_bf16_pages": round(ra_ms / a8_ms, 3)}
            del ctx8, pk8, ws8, kp8, vp8
        del ctx2, pk2, ws2
        # next row: the row pass fused into the LM head GEMM (hidden size of a small dLLM; random inputs)
        hidden = 2048
        gen = torch.Generator(device=dev); gen.manual_seed(seed + 77)
        hx = (torch.randn(rows, hidden, device=dev, generator=gen)).to(torch.bfloat16)
        hw = (torch.randn(wl.vocab, hidden, device=dev, generator=gen) / math.sqrt(hidden)).to(torch.bfloat16)
        lws = torch.zeros(B.lib().fb_lm_head_workspace_bytes(ctx.handle), dtype=torch.uint8, device=dev)
        tok_keep = st.tokens.clone()
        n3 = max(3, min(args.steps, 5))
        ev3 = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(n3)]
        for k in range(2 + n3):
            e = ev3[k - 2] if k >= 2 else None
            if e: e[0].record(stream)
            B.fb_lm_head_t2t(ctx, pk, hx, hw, st, sb.argmax, sb.conf, sb.action, sb.slot_stats, lws, sb.status, stream)
            if e: e[1].record(stream)
        barrier()
        st.tokens.copy_(tok_keep)
        lm_ms = float(np.mean([e[0].elapsed_time(e[1]) for e in ev3]))
        lm_flops = 2.0 * live_now * wl.block_len * wl.vocab * hidden
        nxt["lm_head_t2t"] = {"ms": round(lm_ms, 4), "hidden": hidden, "rows": live_now * wl.block_len,
                              "tflops": round(lm_flops / lm_ms / 1e9, 1),
                              "logits_bytes_not_moved": 2.0 * live_now * wl.block_len * wl.vocab * 2}
        del hx, hw, lws

    # ------------- the same step replayed from a CUDA graph (one graph launch instead of seven launches)
    if only == "all" and world == 1 and not args.no_graph:
        def step_current():
            B.fb_pack_wavefronts(ctx, st, pk, sb.ws, sb.status)
            B.fb_wavefront_attn(ctx, pk, q, kw, vw, kp, vp, st.page_table, sb.out, sb.ws, sb.status)
            B.fb_t2t_step(ctx, pk, logits, st, sb.argmax, sb.conf, sb.action, sb.slot_stats, sb.status)
            B.fb_gate_commit(ctx, pk, sb.slot_stats, st, kw, vw, kp, vp, sb.n_committed, sb.spawned,
                             sb.step_counters, sb.status)
        graph = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        side.wait_stream(stream)
        with torch.cuda.stream(side):
            step_current()                       # per-device set-up already happened: nothing but launches
            side.synchronize()
            with torch.cuda.graph(graph, stream=side):
                step_current()
        stream.wait_stream(side)
        ng = max(3, min(args.steps, 20))
        evg = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(ng)]
        for k in range(3 + ng):
            if flush is not None:
                flush.fill_(k & 0xFF)
            e = evg[k - 3] if k >= 3 else None
            if e: e[0].record(stream)
            graph.replay()
            if e: e[1].record(stream)
        barrier()
        g_ms = [a.elapsed_time(b) for a, b in evg]
        nxt["step_graph_replay"] = {"ms_per_step": round(float(np.mean(g_ms)), 4), "ms_per_step_min": round(float(np.min(g_ms)), 4),
                                    "direct_launch_ms_per_step": round(float(per_step.mean()), 4), "timed_steps": ng,
                                    "device_status": int(sb.status.item())}
        del graph

    # ------------- a step that commits: calibrated confidences, state reset before every timed step
    if only == "all" and world == 1 and not args.no_calibrated:
        nxt["step_calibrated"] = calibrated_step(args, wl, stc_init, dev, stream, q, kw, vw, kp, vp, logits, sb)

    # ------------------------------------------------------------ end to end
    e2e_ms, h2d, d2h = float("nan"), 0, 0
    if not args.no_e2e and only == "all":
        pin = lambda t: t.cpu().contiguous().pin_memory()
        hq, hkw, hvw = pin(q), pin(kw), pin(vw)
        hz = torch.zeros(rows, wl.vocab, dtype=torch.bfloat16).pin_memory()
        hz[:z_live.shape[0]].copy_(z_live)
        host = dict(h_q=hq, h_k_win=hkw, h_v_win=hvw, h_logits=hz,
                    h_n_committed=torch.zeros(wl.n_requests, dtype=torch.int32).pin_memory(),
                    h_spawned=torch.zeros(wl.n_requests, dtype=torch.uint8).pin_memory(),
                    h_step_counters=torch.zeros(B.FB_STEP_COUNTERS, dtype=torch.int32).pin_memory(),
                    h_status=torch.zeros(1, dtype=torch.int32).pin_memory(),
                    n_rows=synth.n_live_slots(stc1) * wl.block_len)
        devb = dict(q=q, k_win=kw, v_win=vw, out=sb.out, logits=logits, k_pool=kp, v_pool=vp,
                    argmax=sb.argmax, conf=sb.conf, action=sb.action, slot_stats=sb.slot_stats,
                    n_committed=sb.n_committed, spawned=sb.spawned, step_counters=sb.step_counters,
                    status=sb.status, ws=sb.ws)
        e2e_steps = max(3, min(args.steps, 5))
        for _ in range(2):
            B.fb_step_host(ctx, st, pk, devb, host, stream)
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(e2e_steps):
            B.fb_step_host(ctx, st, pk, devb, host, stream)
            stream.synchronize()          # the caller reads the step's decisions
        e1.record(stream)
        barrier()
        e2e_ms = e0.elapsed_time(e1) / e2e_steps
        h2d = sum(host["n_rows"] * t[0].numel() * t.element_size() for t in (hq, hkw, hvw, hz))
        d2h = wl.n_requests * 4 + wl.n_requests + B.FB_STEP_COUNTERS * 4 + 4
    t2 = time.time()
    clocks = sampler.stop(t0, t2)
    clocks["window"] = "timed steps + end-to-end steps"

    # algorithmic work of the state the timed steps ran on (mean of the state
    # before and after, equal once the literal-logit workload has settled)
    n_live = (synth.n_live_slots(stc0) + synth.n_live_slots(stc1)) / 2.0
    flops_state = (attn_flops(stc0) + attn_flops(stc1)) / 2.0
    abytes_state = (attn_bytes(stc0) + attn_bytes(stc1)) / 2.0
    stc = stc0
    flops = flops_state
    ms_step = total_ms / args.steps
    (ms_step_max, e2e_ms_max), (flops_all, t2tb_all) = combine_ranks(
        [ms_step, e2e_ms], [flops, t2t_bytes(stc, n_live)], dev, world)
    ranks = gather_ranks({"rank": rank, "device": torch.cuda.get_device_name(local), "uuid": uuid, "seed": seed,
                          "ms_per_step": round(ms_step, 4), "attn_tflop_per_step": round(flops / 1e12, 4)}, world)

    if rank == 0:
        peaks = load_peaks()
        attn_ms, t2t_ms = float(seg[:, 1].mean()), float(seg[:, 2].mean())
        attn_tf = flops / attn_ms / 1e9
        t2t_gbs = t2t_bytes(stc, n_live) / t2t_ms / 1e6
        roof_attn = {"kernel": "wavefront_attn_kernel(+combine)", "bound": "tensor",
                     "achieved": round(attn_tf, 2), "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                     "frac": round(attn_tf / peaks["bf16_tflops"], 4),
                     "traffic": (round(NCU_TRAFFIC_RATIO[("attn", args.workload)] * abytes_state)
                                 if ("attn", args.workload) in NCU_TRAFFIC_RATIO and not args.requests else None),
                     "peak_source": peaks["source"] + " cuBLAS bf16 burst",
                     "hbm_floor_ms": round(abytes_state / peaks["hbm_gbs"] / 1e6, 4),
                     "tensor_floor_ms": round(flops / peaks["bf16_tflops"] / 1e9, 4),
                     "ms": round(attn_ms, 4)}
        roof_t2t = {"kernel": "t2t_rows_kernel(+update)", "bound": "hbm", "achieved": round(t2t_gbs, 1),
                    "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": round(t2t_gbs / peaks["hbm_gbs"], 4),
                    "traffic": (round(NCU_TRAFFIC_RATIO[("t2t", args.workload)] * t2t_bytes(stc, n_live))
                                if ("t2t", args.workload) in NCU_TRAFFIC_RATIO and not args.requests else None),
                    "peak_source": peaks["source"] + " copy bandwidth", "ms": round(t2t_ms, 4)}
        dominant = roof_attn if attn_ms >= t2t_ms else roof_t2t
        line = {
            "metric": METRIC, "value": round(flops_all / ms_step_max / 1e9, 3),
            "unit": "TFLOP/s (attention FLOPs / whole-step time)",
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": round(ms_step_max, 4), "ms_per_step_median": round(float(np.median(per_step)), 4),
            "ms_per_step_min": round(float(per_step.min()), 4), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": wl.name, "requests": wl.n_requests, "block_len": wl.block_len,
                       "wmax": wl.wmax, "slots": ctx.max_slots, "live_slots": n_live, "state_settled": bool(synth.n_live_slots(stc0) == synth.n_live_slots(stc1)),
                       "q_heads": wl.n_q_heads, "kv_heads": wl.n_kv_heads, "head_dim": wl.head_dim,
                       "vocab": wl.vocab, "prefix_range": [wl.prefix_lo, wl.prefix_hi],
                       "logits": wl.logits_kind, "parallelism": f"replicas x{world}",
                       "l2": ("inputs larger than L2 (logits + KV pools >> 126 MB); no flush" if flush is None else
                              "inputs fit in L2: a 256 MB write between the timed steps evicts them")},
            "clocks": clocks,
            "e2e": {"value": round(flops_all / e2e_ms_max / 1e9, 3),
                    "unit": "TFLOP/s (attention FLOPs / whole-step time)", "buffers": "host (pinned)",
                    "ms_per_step": round(e2e_ms_max, 3), "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h,
                    "t2t_gbs": round(t2tb_all / e2e_ms_max / 1e6, 2)},
            "gpu_launches": KERNELS_PER_STEP * args.steps,
            "kernels": {"pack_ms": round(float(seg[:, 0].mean()), 4), "attn_ms": round(attn_ms, 4),
                        "t2t_ms": round(t2t_ms, 4), "gate_commit_ms": round(float(seg[:, 3].mean()), 4),
                        "attn_tflops": round(attn_tf, 2), "t2t_gbs": round(t2t_gbs, 1),
                        "attn_frac_of_nominal_2250": round(attn_tf / 2250.0, 4),
                        "t2t_frac_of_nominal_8000": round(t2t_gbs / 8000.0, 4)},
            "roofline": {k: dominant[k] for k in ("bound", "achieved", "peak", "unit", "frac", "traffic")}
                        | {"kernel": dominant["kernel"], "peak_source": dominant["peak_source"]},
            "roofline_attn": roof_attn, "roofline_t2t": roof_t2t,
            "device_status": status, "step_counters": counters,
            "ranks": ranks,
        }
        if nxt:
            nxt["lm_head_t2t"]["frac_of_measured_bf16"] = round(nxt["lm_head_t2t"]["tflops"] / peaks["bf16_tflops"], 4)
            nxt["scatter_window_kv"]["frac_of_measured_hbm"] = round(nxt["scatter_window_kv"]["gbs"] / peaks["hbm_gbs"], 4)
            f8 = nxt.get("attn_fp8_pages", {})
            f8["peak_fp8_tflops"] = round(2.0 * peaks["bf16_tflops"], 1)      # measured bf16 burst x the nominal fp8 : bf16 ratio (4.5 : 2.25)
            if "tflops" in f8:
                f8["frac_of_fp8_peak"] = round(f8["tflops"] / f8["peak_fp8_tflops"], 4)
                f8["hbm_floor_ms"] = round(f8["algorithmic_bytes"] / peaks["hbm_gbs"] / 1e6, 4)
            line["next_rows"] = nxt
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(wl, stc_init, tokens, z_live, attn, budget_s=args.cpu_budget)
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def calibrated_step(args, wl, stc, dev, stream, q, kw, vw, kp, vp, logits, sb):
    """The bench workload's structure with confidence-calibrated logits (winner
    confidences U(0.8, 0.999) on 70 % of the rows) and S_pe = 0, the initial
    state restored before every timed step: each timed step reveals, edits,
    retires blocks (KV freeze copy of Eq. 6) and admits new ones.  Device time
    of the four calls by CUDA events; the logits of the main run are
    overwritten."""
    import torch
    from paper_2607_17652_b200 import binding as B, synth
    tokens0 = synth.make_tokens(stc)
    n_live = synth.n_live_slots(stc)
    z, tokens0 = synth.make_logits(stc, tokens0, "calibrated", conf_shift=0.3, n_rows=n_live * wl.block_len)
    logits[:z.shape[0]].copy_(z)
    ctx = B.Context(**synth.config_dict(stc, s_pe=0))
    st = B.DeviceState.from_numpy(dev, stc.active, stc.prefix_len, stc.L, stc.R, tokens0,
                                  np.zeros((wl.n_requests, wl.wmax), np.uint8), stc.page_table)
    snap = {k: getattr(st, k).clone() for k in ("active", "prefix_len", "L", "R", "tokens", "pe_done")}
    pk = B.PackBuffers.alloc(ctx, dev)
    ws = B.alloc_workspace(ctx, dev)
    n = max(3, min(args.steps, 10))
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(n)]
    for k in range(3 + n):
        for name, v in snap.items():
            getattr(st, name).copy_(v)
        e = evs[k - 3] if k >= 3 else None
        if e: e[0].record(stream)
        B.fb_pack_wavefronts(ctx, st, pk, ws, sb.status, stream)
        if e: e[1].record(stream)
        B.fb_wavefront_attn(ctx, pk, q, kw, vw, kp, vp, st.page_table, sb.out, ws, sb.status, stream)
        if e: e[2].record(stream)
        B.fb_t2t_step(ctx, pk, logits, st, sb.argmax, sb.conf, sb.action, sb.slot_stats, sb.status, stream)
        if e: e[3].record(stream)
        B.fb_gate_commit(ctx, pk, sb.slot_stats, st, kw, vw, kp, vp, sb.n_committed, sb.spawned,
                         sb.step_counters, sb.status, stream)
        if e: e[4].record(stream)
    torch.cuda.synchronize()
    seg = np.array([[e[i].elapsed_time(e[i + 1]) for i in range(4)] for e in evs]).mean(0)
    c = sb.step_counters.cpu().numpy().tolist()
    blocks = c[0]
    freeze_bytes = 2.0 * 2 * blocks * wl.block_len * wl.n_kv_heads * wl.head_dim * 2      # K and V, read + write
    return {"ms": round(float(seg.sum()), 4), "pack_ms": round(float(seg[0]), 4), "attn_ms": round(float(seg[1]), 4),
            "t2t_ms": round(float(seg[2]), 4), "gate_commit_ms": round(float(seg[3]), 4),
            "attn_tflops": round(attn_flops(stc) / float(seg[1]) / 1e9, 2),
            "t2t_gbs": round(t2t_bytes(stc, n_live) / float(seg[2]) / 1e6, 1),
            "committed_blocks_per_step": blocks, "committed_tokens_per_step": c[1], "spawned_per_step": c[2],
            "reveals_per_step": c[4], "edits_per_step": c[5], "finished_requests_per_step": c[3],
            "kv_freeze_bytes": freeze_bytes, "kv_freeze_gbs": round(freeze_bytes / float(seg[3]) / 1e6, 1),
            "logits": "calibrated (+0.3)", "s_pe": 0, "state": "initial state restored before every timed step",
            "timed_steps": n, "device_status": int(sb.status.item())}


# ------------------------------------------------------------ serving sweep
def run_sweep(args):
    """`--sweep`: the serving workload as a sequence -- requests arrive over the
    first 24 steps, confidences rise by 0.05 per step, blocks reveal, commit and
    spawn (48 steps by default).  One untimed pass, then the timed one; every
    step's four calls are bracketed by CUDA events, logits patching (it stands
    in for the LM head) stays outside.  Reports steps/s and committed tokens/s
    beside the usual fields; the rows that are live come from the device state
    read back before each step."""
    import dataclasses
    import torch
    from paper_2607_17652_b200 import binding as B, sweep, synth
    B.lib()                                     # fails loudly when the CUDA library is missing
    dev = "cuda:0"
    torch.cuda.set_device(0)
    wl = synth.WORKLOADS[args.workload]
    if args.requests:
        wl = dataclasses.replace(wl, n_requests=args.requests)
    over = {}
    if args.wmax:
        over["wmax"] = args.wmax
    if args.theta is not None:
        over["theta_spawn"] = args.theta
    if args.block_len:
        over["block_len"] = args.block_len
        over["max_blocks"] = max(2, wl.max_blocks * wl.block_len // args.block_len)
    wl = dataclasses.replace(wl, **over)
    n_steps = args.steps if args.steps != 20 else 48
    rise = tuple(float(x) for x in args.rise_range.split(",")) if args.rise_range else None
    inp = sweep.SweepInputs(wl, n_steps=n_steps, arrive_hi=1 if args.static_batch else 24, rise_range=rise)
    run = sweep.SweepRunner(inp, dev, window_in_pages=args.window_in_pages, batch_sync=args.batch_sync,
                            kv_fp8=args.kv_fp8)

    def one_pass(timed):
        seg, flops, live, committed = [], [], [], 0
        for step in range(n_steps):
            for r in inp.arrivals(step):
                run.arrive(r)
            active, plen, L, R = run.host_state()
            rows, cols, vals, _ = inp.begin_step(step, active, L, R)
            inp.apply(run.z, rows, cols, vals)
            cur = dataclasses.replace(inp.stc)
            cur.active, cur.prefix_len, cur.L, cur.R = active, plen, L, R
            t = run.step()
            if timed:
                seg.append(t)
                flops.append(attn_flops(cur))
                live.append(len(rows) // wl.block_len)
                committed += int(run.sb.n_committed.sum().item()) * wl.block_len
        return np.array(seg), np.array(flops), np.array(live), committed

    one_pass(False)
    run.reset()
    uuid = str(torch.cuda.get_device_properties(0).uuid)
    sampler = ClockSampler(uuid if uuid.startswith("GPU-") else "GPU-" + uuid)
    sampler.start()
    time.sleep(0.2)
    t0 = time.time()
    seg, flops, live, committed = one_pass(True)
    t1 = time.time()
    clocks = sampler.stop(t0, t1)
    clocks["window"] = "the timed pass of the sweep (device time is a fraction of it: inputs are patched between steps)"
    status = int(run.sb.status.item())
    total_ms = float(seg.sum())
    peaks = load_peaks()
    attn_ms, t2t_ms = float(seg[:, 1].sum()), float(seg[:, 2].sum())
    attn_tf = float(flops.sum()) / attn_ms / 1e9
    t2t_b = float(sum(l * wl.block_len * (2.0 * wl.vocab + 13) + l * 24 for l in live))
    t2t_gbs = t2t_b / t2t_ms / 1e6
    line = {
        "metric": METRIC, "value": round(float(flops.sum()) / total_ms / 1e9, 3),
        "unit": "TFLOP/s (attention FLOPs / whole-step time)",
        "n_gpus": 1, "steps": n_steps, "warmup": n_steps, "ms_per_step": round(total_ms / n_steps, 4),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "fp8 e4m3 (K/V pages, Q, P; fp32 accumulation)" if args.kv_fp8 else "bf16", "data": "synthetic",
        "config": {"workload": wl.name + (" (sweep, FP8 E4M3 pages)" if args.kv_fp8 else
                                          " (sweep, window in pages)" if args.window_in_pages else " (sweep)"), "requests": wl.n_requests, "block_len": wl.block_len,
                   "wmax": wl.wmax, "theta_spawn": wl.theta_spawn,
                   "policy": "batch-synchronous wavefront" if args.batch_sync else "per-sequence wavefronts",
                   "arrivals": "all at step 0" if args.static_batch else "uniform over the first 24 steps",
                   "confidence_rise_per_step": list(rise) if rise else 0.05,
                   "slots": wl.max_slots, "live_slots": float(live.mean()),
                   "q_heads": wl.n_q_heads, "kv_heads": wl.n_kv_heads, "head_dim": wl.head_dim,
                   "vocab": wl.vocab, "prefix_range": [wl.prefix_lo, wl.prefix_hi],
                   "logits": "noise bank, one winner per live row patched per step", "parallelism": "replicas x1",
                   "l2": "inputs larger than L2 (logits + KV pools >> 126 MB); no flush"},
        "sweep": {"steps_per_s": round(n_steps / total_ms * 1e3, 1),
                  "committed_tokens_per_s": round(committed / total_ms * 1e3, 1),
                  "committed_tokens": committed, "committed_tokens_per_step": round(committed / n_steps, 2),
                  "live_slots_first_last": [int(live[0]), int(live[-1])],
                  "device_ms_total": round(total_ms, 3)},
        "clocks": clocks,
        "e2e": {"value": None, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0,
                "note": "the sweep is timed with resident inputs only; see the default run for host buffers"},
        "gpu_launches": KERNELS_PER_STEP * n_steps,
        "kernels": {"pack_ms": round(float(seg[:, 0].mean()), 4), "attn_ms": round(attn_ms / n_steps, 4),
                    "t2t_ms": round(t2t_ms / n_steps, 4), "gate_commit_ms": round(float(seg[:, 3].mean()), 4),
                    "attn_tflops": round(attn_tf, 2), "t2t_gbs": round(t2t_gbs, 1)},
        "roofline": {"bound": "tensor", "achieved": round(attn_tf, 2), "peak": peaks["bf16_tflops"],
                     "unit": "TFLOP/s", "frac": round(attn_tf / peaks["bf16_tflops"], 4), "traffic": None,
                     "kernel": "wavefront_attn_kernel(+combine)",
                     "peak_source": peaks["source"] + " cuBLAS bf16 burst"},
        "roofline_t2t": {"bound": "hbm", "achieved": round(t2t_gbs, 1), "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": round(t2t_gbs / peaks["hbm_gbs"], 4), "traffic": None},
        "device_status": status,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------- the oracle, timed
def oracle_sample_step(wl, stc, tokens, z_live, attn, n_req):
    """One oracle step (pack, attention, T2T, gate/commit) on the first n_req
    decoding requests of the workload.  Returns (seconds, attention flops,
    slots, rows)."""
    from oracle import flowblock_oracle as O
    from tests import harness as H
    keep = np.flatnonzero(stc.active == 1)[:n_req]
    sp = H.sub_problem(stc, tokens, attn, z_live, keep)
    ocfg, ost, sub = sp["ocfg"], sp["ost"], sp["sub"]
    fq, fkw, fvw, fkp, fvp, fz = sp["q"], sp["k_win"], sp["v_win"], sp["k_pool"], sp["v_pool"], sp["logits"]
    b = wl.block_len
    t0 = time.perf_counter()
    opk = O.pack_wavefronts(ocfg, ost)
    O.wavefront_attn(ocfg, opk, fq, fkw, fvw, fkp, fvp, ost.page_table)
    xhat, conf = O.t2t_rows(ocfg, opk, fz)
    action, stats = O.t2t_update(ocfg, opk, ost, xhat, conf)
    O.gate_commit(ocfg, opk, stats, ost, fkw, fvw, fkp, fvp)
    dt = time.perf_counter() - t0
    return dt, attn_flops(sub), opk.n_live, opk.n_live * b


def cpu_baseline(wl, stc, tokens, z_live, attn, budget_s=12.0):
    n_req, used = 1, None
    total = int((stc.active == 1).sum())
    while True:
        dt, fl, slots, rows = oracle_sample_step(wl, stc, tokens, z_live, attn, n_req)
        used = (dt, fl, slots, rows, n_req)
        if dt >= budget_s or n_req >= total:
            break
        n_req = min(total, max(n_req + 1, int(n_req * min(4.0, budget_s / max(dt, 1e-3)))))
    dt, fl, slots, rows, n_req = used
    try:
        import threadpoolctl
        threads = max([p["num_threads"] for p in threadpoolctl.threadpool_info()] or [1])
    except Exception:
        threads = os.cpu_count()
    return {"value": round(fl / dt / 1e12, 6), "unit": "TFLOP/s (attention FLOPs / whole-step time)",
            "cores": threads, "host_cores": os.cpu_count(), "kind": "oracle", "seconds": round(dt, 2),
            "sample": f"first {n_req} of {total} requests of {wl.name}: {slots} slots, {rows} rows x V={wl.vocab}"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2607_17652_b200 import synth
    wl = pick_workload(args)
    stc, tokens, n_live, z_live, attn = build_inputs(wl, synth.BASE_SEED + wl.index)
    n_req = args.ref_requests
    times, fl = [], 0.0
    for k in range(args.warmup + args.steps):
        dt, fl, slots, rows = oracle_sample_step(wl, stc, tokens, z_live, attn, n_req)
        if k >= args.warmup:
            times.append(dt)
    ms = 1e3 * sum(times) / len(times)
    val = round(fl / (ms / 1e3) / 1e12, 6)
    unit = "TFLOP/s (attention FLOPs / whole-step time)"
    try:
        import threadpoolctl
        threads = max([p["num_threads"] for p in threadpoolctl.threadpool_info()] or [1])
    except Exception:
        threads = os.cpu_count()
    total = int((stc.active == 1).sum())
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": unit,
            "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": round(ms, 3), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic",
            "config": {"workload": wl.name, "requests": wl.n_requests, "block_len": wl.block_len,
                       "wmax": wl.wmax, "vocab": wl.vocab},
            "cpu_baseline": {"value": val, "unit": unit, "kind": "oracle", "cores": threads,
                             "host_cores": os.cpu_count(),
                             "sample": f"each step: first {n_req} of {total} requests of {wl.name}: "
                                       f"{slots} slots, {rows} rows x V={wl.vocab}"},
            "e2e": {"value": val, "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=DEFAULT_WORKLOAD)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-calibrated", action="store_true", help="skip next_rows.step_calibrated")
    ap.add_argument("--no-graph", action="store_true", help="skip next_rows.step_graph_replay")
    ap.add_argument("--target-items", type=int, default=0, help="fb_tuning.attn_target_items (0: default)")
    ap.add_argument("--min-chunk", type=int, default=0, help="fb_tuning.attn_min_chunk_tiles (0: default)")
    ap.add_argument("--pair", action="store_true",
                    help="quads of Q tiles on the CTA-pair attention kernel (fb_tuning.attn_pair): the comparison run")
    ap.add_argument("--dry-run-cpu", action="store_true",
                    help="launcher / reduction plumbing only: gloo ranks on CPU, no kernel, placeholder times")
    ap.add_argument("--requests", type=int, default=0,
                    help="override the workload's request count (small cases for profiler captures)")
    ap.add_argument("--only", default="all", choices=["all", "attn", "t2t", "attn_fp8"],
                    help="time one call only (profiler captures); the JSON line then has no step metric")
    ap.add_argument("--cpu-budget", type=float, default=12.0)
    ap.add_argument("--ref-requests", type=int, default=2)
    ap.add_argument("--window-in-pages", action="store_true",
                    help="with --sweep: scatter the window K/V into the pages every step (Eq. 6), attention "
                         "over the pages, retirement as a pointer bump")
    ap.add_argument("--kv-fp8", action="store_true",
                    help="with --sweep: KV pages in FP8 E4M3 (scatter = quantiser every step, 8-bit attention products)")
    ap.add_argument("--batch-sync", action="store_true",
                    help="with --sweep: the batch-synchronous wavefront of the packing ablation (fb_config.batch_sync)")
    ap.add_argument("--static-batch", action="store_true", help="with --sweep: every request arrives at step 0")
    ap.add_argument("--rise-range", default="",
                    help="with --sweep: lo,hi of the per-request confidence rise per step (default 0.05 for all)")
    ap.add_argument("--wmax", type=int, default=0, help="with --sweep: window bound W")
    ap.add_argument("--theta", type=float, default=None, help="with --sweep: admission gate theta_spawn")
    ap.add_argument("--block-len", type=int, default=0, help="with --sweep: block length bl")
    ap.add_argument("--sweep", action="store_true",
                    help="run the serving workload as a 48-step sequence with arrivals (use with --workload 4)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours":
        sys.exit(launch_replicas(args))
    if args.impl == "reference":
        run_reference(args)
    elif args.dry_run_cpu:
        run_dry(args)
    elif args.only == "attn_fp8":
        run_fp8_only(args)
    elif args.sweep:
        run_sweep(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
