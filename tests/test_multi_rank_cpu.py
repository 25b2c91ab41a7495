"""World-size-2 gloo test (CPU) of the host logic behind `bench.py --gpus N`: rows are independent, so every rank
takes its own block of rows, there is no data-path collective, and the only exchange is the max over ranks of the
timing.  The per-rank blocks must tile the workload exactly and regenerate bit-identically from (seed, index)."""
from __future__ import annotations

import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2512_09196_b200 import inputs


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = inputs.Workload("t", "layernorm", inputs.BF16, 37, 64, seed=5, x_mean=0.5, x_std=3.0, eps=1e-5)
    row0, n = inputs.shard_rows(w.rows, rank, world)
    x = w.generate(row0, n)["x"]
    # what bench.py exchanges: each rank's elapsed time, reduced with MAX
    t = torch.tensor([10.0 + rank], dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    checksum = torch.tensor([int(x.astype(np.uint64).sum()), n], dtype=torch.int64)
    gathered = [torch.zeros(2, dtype=torch.int64) for _ in range(world)]
    dist.all_gather(gathered, checksum)
    if rank == 0:
        out.put((float(t.item()), [g.tolist() for g in gathered]))
    dist.barrier()
    dist.destroy_process_group()


def test_row_sharding_over_two_gloo_ranks():
    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    tmax, gathered = q.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert tmax == 11.0                                   # max over ranks, not rank 0's own time
    full = inputs.Workload("t", "layernorm", inputs.BF16, 37, 64, seed=5, x_mean=0.5, x_std=3.0, eps=1e-5).generate()["x"]
    assert sum(n for _, n in gathered) == 37
    pos = 0
    for s, n in gathered:
        assert s == int(full[pos:pos + n].astype(np.uint64).sum())
        pos += n
