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
