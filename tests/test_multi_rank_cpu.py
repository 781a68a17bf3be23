"""The N > 1 path of the benchmark on CPU: two gloo ranks, each with its own circuit (weak scaling, no collective
on the data path).  Checks the only cross-rank logic there is -- whole-job time is the maximum over ranks, work
is the sum -- and that ranks draw different circuits of the same shape."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench
from paper_2502_01681_b200 import synth


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = synth.workload(5, 2000)
    w.seed = w.seed + 1000 * rank                      # as bench.py does per rank
    g = w.graph()
    seconds = 0.5 + 0.25 * rank                        # rank 1 is the slow one
    t, u = bench.reduce_over_ranks(dist, "cpu", seconds, g.n * 6)
    out.put((rank, g.n, int(g.col_idx[:64].sum()), t, u))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_reduce_time_by_max_and_work_by_sum():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, n0, sig0, t0, u0), (r1, n1, sig1, t1, u1) = res
    assert n0 == n1 and sig0 != sig1                   # same shape, different circuits
    assert t0 == t1 == 0.75                            # max over ranks
    assert u0 == u1 == (n0 + n1) * 6                   # sum over ranks


def test_single_process_passes_through():
    assert bench.reduce_over_ranks(None, "cpu", 1.5, 10) == (1.5, 10.0)
