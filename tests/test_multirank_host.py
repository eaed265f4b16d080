"""The N > 1 path of the benchmark, host side, on CPU: two `gloo` ranks draw batches of their own,
sum their parameter gradients with one all-reduce and report the whole job as (sum of units) /
(max of times).  The device path itself needs no collective: instances never exchange tokens."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    import bench
    import workloads
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        seed = bench.rank_seed(workloads.DEFAULT_SEED, rank)
        cfg = workloads.config(3, seed=seed, B=16, V=50, H=8)
        n = cfg["trees"].N
        grads = {"W": torch.full((2, 3), float(rank + 1)), "b": torch.arange(3, dtype=torch.float32) * (rank + 1)}
        bench.sum_gradients(dist, grads)
        elapsed, units = bench.reduce_job(dist, "cpu", 10.0 + rank, n)
        out.put((rank, seed, n, elapsed, units, grads["W"].tolist(), grads["b"].tolist()))
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_instances_and_sum_gradients():
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
    (r0, s0, n0, t0, u0, w0, b0), (r1, s1, n1, t1, u1, w1, b1) = res
    assert s0 != s1                                   # every rank has a batch of its own
    assert t0 == t1 == 11.0                           # time of the job = the slowest rank
    assert u0 == u1 == n0 + n1                        # units of the job = all ranks' invocations
    assert w0 == w1 == np.full((2, 3), 3.0).tolist()  # 1 + 2
    assert b0 == b1 == [0.0, 3.0, 6.0]


def test_single_rank_needs_no_process_group():
    import bench
    assert bench.reduce_job(None, "cpu", 5.0, 123) == (5.0, 123.0)
    g = {"W": torch.ones(2)}
    bench.sum_gradients(None, g)
    assert g["W"].tolist() == [1.0, 1.0]
