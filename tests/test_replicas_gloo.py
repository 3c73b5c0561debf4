"""The N > 1 path on CPU: two gloo ranks run the replica bookkeeping the benchmark uses
(per-rank seeds, time = max over ranks, job throughput = all ranks' units / that time)."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2602_02864_b200 import replicas, workloads as wl


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert replicas.rank_and_world() == (rank, world)
        # every rank draws its own scenes: same recipe, different values
        w = wl.cfg2_batched(layers=1, batch=2)
        g = torch.Generator().manual_seed(w.seed + 7919 * replicas.replica_seed_shift(rank))
        first = float(torch.randn(4, generator=g)[0])
        # rank r "measures" (r + 1) * 10 ms over 1000 units
        ms = 10.0 * (rank + 1)
        tput, job_ms = replicas.job_throughput(1000.0, ms)
        replicas.barrier()
        out.put((rank, first, replicas.max_over_ranks(ms), replicas.sum_over_ranks(1.0), tput, job_ms))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_aggregate_like_the_benchmark():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res[0][1] != res[1][1]                       # different scenes per rank
    for rank, _, mx, cnt, tput, job_ms in res:
        assert mx == 20.0 and job_ms == 20.0            # the slowest rank's time
        assert cnt == 2.0
        assert np.isclose(tput, 2000.0 / 20e-3)         # all ranks' units over the job time


def test_single_process_is_identity():
    assert replicas.rank_and_world() == (0, 1)
    assert replicas.max_over_ranks(3.5) == 3.5
    tput, ms = replicas.job_throughput(100.0, 50.0)
    assert ms == 50.0 and np.isclose(tput, 2000.0)
