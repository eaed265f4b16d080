"""The N > 1 path of the benchmark, host side, on CPU: `bench.spawn_ranks` starts two ranks (the path that
`bench.py --gpus N` takes when no launcher provided them), which join a `gloo` group, draw batches of their
own, sum their parameter gradients with ONE all-reduce over the flat gradient buffer and report the whole job
as (sum of units) / (max of times).  The device path itself needs no collective: instances never exchange tokens."""
import json
import os
import sys

import numpy as np
import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _gloo_rank(payload):
    """What one rank does (module level: the spawned processes import it by name)."""
    import torch.distributed as dist

    import bench
    import workloads
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    assert int(os.environ["LOCAL_RANK"]) == rank and os.environ["MASTER_ADDR"] == "127.0.0.1"
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        seed = bench.rank_seed(workloads.DEFAULT_SEED, rank)
        cfg = workloads.config(3, seed=seed, B=16, V=50, H=8)
        n = cfg["trees"].N
        flat, grads = bench.flat_gradients({"W": (2, 3), "b": (3,)}, "cpu")
        grads["W"].fill_(float(rank + 1))
        grads["b"].copy_(torch.arange(3, dtype=torch.float32) * (rank + 1))
        calls = []
        real = dist.all_reduce
        dist.all_reduce = lambda t, *a, **k: (calls.append(t.numel()), real(t, *a, **k))[1]
        bench.sum_gradients(dist, flat)
        dist.all_reduce = real
        elapsed, units = bench.reduce_job(dist, "cpu", 10.0 + rank, n)
        with open(os.path.join(payload["dir"], f"rank{rank}.json"), "w") as f:
            json.dump({"rank": rank, "seed": seed, "n": n, "elapsed": elapsed, "units": units, "W": grads["W"].tolist(),
                       "b": grads["b"].tolist(), "all_reduce_calls": calls, "flat": flat.numel()}, f)
    finally:
        dist.destroy_process_group()


def _failing_rank(payload):
    if os.environ["RANK"] == "1":
        raise RuntimeError("rank 1 fails on purpose")


def test_spawned_ranks_shard_instances_and_sum_gradients(tmp_path):
    import bench
    bench.spawn_ranks(2, _gloo_rank, {"dir": str(tmp_path)})
    r0, r1 = (json.load(open(tmp_path / f"rank{r}.json")) for r in range(2))
    assert r0["seed"] != r1["seed"]                               # every rank has a batch of its own
    assert r0["elapsed"] == r1["elapsed"] == 11.0                 # time of the job = the slowest rank
    assert r0["units"] == r1["units"] == r0["n"] + r1["n"]        # units of the job = all ranks' invocations
    assert r0["W"] == r1["W"] == np.full((2, 3), 3.0).tolist()    # 1 + 2
    assert r0["b"] == r1["b"] == [0.0, 3.0, 6.0]
    assert r0["all_reduce_calls"] == [r0["flat"]]                 # one collective for all gradients


def test_a_failing_rank_fails_the_launch():
    import bench
    with pytest.raises(Exception):
        bench.spawn_ranks(2, _failing_rank, {})


def test_flat_gradient_views_are_aligned_and_disjoint():
    import bench
    flat, g = bench.flat_gradients({"E": (7, 5), "W": (3, 6), "b": (3,)}, "cpu")
    for k, v in g.items():
        assert (v.data_ptr() - flat.data_ptr()) % 256 == 0
        v.fill_(1.0)
    assert flat.sum().item() == 35 + 18 + 3


def test_single_rank_needs_no_process_group():
    import bench
    assert bench.reduce_job(None, "cpu", 5.0, 123) == (5.0, 123.0)
    g = {"W": torch.ones(2)}
    bench.sum_gradients(None, g)
    assert g["W"].tolist() == [1.0, 1.0]


def test_asking_for_more_gpus_than_present_is_refused():
    """`--gpus N` never reports fewer GPUs than asked: without N devices (none on a CPU machine) it exits with an error."""
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "64", "--steps", "1"], env=env,
                       capture_output=True, text=True, timeout=300)
    assert r.returncode != 0 and "--gpus 64" in (r.stderr + r.stdout)
