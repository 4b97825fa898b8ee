"""The path shards without any exchange step (independent samples, replicated
weights): N ranks are N replicas. These world-size-2 gloo runs cover the host
logic a multi-GPU bench relies on: per-rank seeded batches are disjoint draws,
max-over-ranks timing, and rank 0 alone reporting."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2212_01005_b200 import workloads as WL


def _free_port():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); p = s.getsockname()[1]; s.close()
    return p


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = WL.mbv2_block("t", [3], 2, 6, 8, 16, 8, 1, True)
    d = WL.generate(wl, list(wl.seed_seq) + [1000 + 10000 * rank])       # the bench's per-rank seed recipe
    digest = torch.tensor([float(np.abs(d["inputs"][0]).sum())], dtype=torch.float64)
    gathered = [torch.zeros(1, dtype=torch.float64) for _ in range(world)]
    dist.all_gather(gathered, digest)
    ms = torch.tensor([1.0 + rank], dtype=torch.float64)                   # rank 1 is the slow one
    dist.all_reduce(ms, op=dist.ReduceOp.MAX)
    samples = torch.tensor([float(wl.samples)], dtype=torch.float64)
    dist.all_reduce(samples, op=dist.ReduceOp.SUM)
    dist.barrier()
    if rank == 0:
        out.put(([float(g.item()) for g in gathered], float(ms.item()), float(samples.item())))
    dist.destroy_process_group()


def test_two_replicas_draw_different_batches_and_time_is_max_over_ranks():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    digests, ms, samples = q.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert digests[0] != digests[1]            # each replica works on its own batch (weak scaling)
    assert ms == 2.0                           # the slowest rank sets the step time
    assert samples == 4.0                      # whole-job samples = sum over replicas
