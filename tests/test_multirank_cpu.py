"""The N > 1 path of the benchmark on CPU (gloo, world size 2): ranks are
independent replicas, so the only cross-rank logic is the MAX-of-times /
SUM-of-work reduction and rank-dependent input seeds."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2607_17652_b200 import synth
    wl = synth.tiny_workload()
    stc = synth.make_structure(wl, synth.BASE_SEED + 1000 * rank)      # each rank its own batch
    flops = bench.attn_flops(stc)
    times, work = bench.combine_ranks([1.0 + rank, 10.0 - rank], [flops, 100.0 * (rank + 1)], "cpu", world)
    out.put((rank, times, work, flops, stc.prefix_len.tolist()))
    dist.barrier()
    dist.destroy_process_group()


def test_replica_reduction_world_size_2():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, t0, w0, f0, p0), (r1, t1, w1, f1, p1) = res
    assert t0 == t1 == [2.0, 10.0]                       # max over ranks
    assert w0 == w1 and abs(w0[0] - (f0 + f1)) < 1e-6 and w0[1] == 300.0   # sum over ranks
    assert p0 != p1                                      # different batches per rank


def test_flop_and_byte_counts_match_definition():
    import bench
    from paper_2607_17652_b200 import synth
    wl = synth.WORKLOADS[1]
    stc = synth.make_structure(wl)
    tot = 0
    for r in range(wl.n_requests):
        for s in range(int(stc.R[r] - stc.L[r])):
            kv_len = int(stc.prefix_len[r]) + (s + 1) * wl.block_len
            tot += 4 * wl.head_dim * wl.block_len * wl.n_q_heads * kv_len   # QK^T and PV, 2 flops per MAC
    assert bench.attn_flops(stc) == float(tot)
    n_live = synth.n_live_slots(stc)
    assert bench.t2t_bytes(stc, n_live) >= n_live * wl.block_len * wl.vocab * 2


def _run_bench(*flags):
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items()
           if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--dry-run-cpu", *flags],
                       capture_output=True, text=True, timeout=300, env=env, cwd=root)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, r.stdout                       # rank 0 alone prints, one line
    return json.loads(lines[0])


def test_bench_starts_its_own_replicas_for_gpus_2():
    """`python bench.py --gpus 2` with no launcher around it starts two ranks
    itself (here over gloo, with the CUDA step left out): the line says two
    GPUs, the ranks drew different batches, times are the MAX and work the SUM
    over them."""
    two = _run_bench("--gpus", "2")
    assert two["n_gpus"] == 2 and two["config"]["parallelism"] == "replicas x2"
    assert [r["rank"] for r in two["ranks"]] == [0, 1]
    assert two["ranks"][0]["seed"] + 1000 == two["ranks"][1]["seed"]
    assert two["ms_per_step"] == 2.0 and two["e2e"]["ms_per_step"] == 11.0
    total = sum(r["attn_flops"] for r in two["ranks"])
    assert abs(two["value"] - total / 2.0 / 1e9) < 1e-9 * total
    one = _run_bench()
    assert one["n_gpus"] == 1 and one["config"]["parallelism"] == "replicas x1"
    assert one["ms_per_step"] == 1.0 and len(one["ranks"]) == 1
