"""GPU parity, recursion shaped by the values it computes (Section 6.2, last paragraph): a tree is grown top-down
from a seed state, a gate on every node's state decides whether the node is expanded.  The CUDA executor
(token waves and vector operators interleaved, through the C boundary) against the fp64 oracle: the state of every
generated tree's root, and the shape of every generated tree (invocations per function, read off the Call records).
The gate is a sign decision on an fp32 sum: an instance whose nearest decision is closer to zero than 1e-4 in the
oracle may legitimately grow a different tree in fp32; such instances are only required to be few, the others must
agree in shape exactly and in value within the fp32 tolerance."""
import numpy as np
import pytest

import workloads
import paper_2410_20225_b200 as rdf
from oracle import direct

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

MARGIN = 1e-4
TOL = 1e-4


def oracle_run(P, tb, D):
    states, logs = [], []
    for b in range(tb.B):
        log = {}
        states.append(direct.topdown(P, int(tb.tok[b]), D, log))
        logs.append(log)
    return np.array(states), logs


def shapes_from_trace(tr, B, n_frames):
    """Per instance: number of Call firings per callee-site label, from the (frame, parent, label) records."""
    calls = tr[tr["kind"] == 0]
    frame = calls["tag"].astype(np.int64) & 0xFFFFFFFF
    parent = np.full(n_frames, -1, dtype=np.int64)
    parent[frame] = calls["parent"]
    inst = np.arange(n_frames, dtype=np.int64)
    inst[B:] = -1
    order = np.sort(frame)                       # frame ids grow with the wave: a parent has a smaller id than its callee
    for f in order:
        inst[f] = inst[parent[f]]
    per = {}
    for f, l in zip(frame, calls["label"]):
        per.setdefault(int(inst[f]), {}).setdefault(int(l), 0)
        per[int(inst[f])][int(l)] += 1
    return per


@pytest.mark.parametrize("H,D,B", [(64, 8, 256), (100, 6, 96), (256, 7, 64), (8, 10, 33)])
def test_topdown_recursion_states_and_shapes(H, D, B):
    V = 1000
    P = workloads.topdown_params(workloads.DEFAULT_SEED + H, V, H)
    tb = workloads.topdown_batch(workloads.DEFAULT_SEED + H, B, V)
    want, logs = oracle_run(P, tb, D)
    total = sum(1 + l["expand"] + l["child"] for l in logs)
    fs, r = rdf.topdown_program(D)
    g = rdf.Graph(fs, r, rdf.TAGS_FRAME)
    h, tr = g.eval_trees(rdf.Graph.device_trees(tb), rdf.Graph.device_params(P), rdf.F32, trace_capacity=4 * total + 64,
                         max_invocations=2 * total + 64)
    h = h.cpu().numpy()
    st = g.stats()
    decisive = np.array([l["margin"] > MARGIN for l in logs])
    assert decisive.mean() >= 0.9, decisive.mean()
    # shapes: per instance, one seed call, `expand` calls over its three sites, left and right calls
    per = shapes_from_trace(tr, B, B + 2 * total + 64)
    for b in np.flatnonzero(decisive):
        n_calls = sum(per[b].values())
        assert n_calls == 1 + logs[b]["expand"] + logs[b]["child"], (b, per[b], logs[b])
    if decisive.all():
        assert st["invocations"] == total
    # values
    err = np.abs(h[decisive] - want[decisive]).max() / np.abs(want[decisive]).max()
    assert err <= TOL, err
    # the generated trees differ in size across the batch: the control really followed the values
    assert len({l["expand"] for l in logs}) >= 4


def test_topdown_degenerate_gates():
    """Gate always open: every tree is the seed alone (three invocations: seed, expand, and nothing below).  Gate
    never open: the full tree down to the depth limit."""
    V, H, D, B = 50, 16, 4, 40
    P = workloads.topdown_params(7, V, H)
    tb = workloads.topdown_batch(7, B, V)
    fs, r = rdf.topdown_program(D)
    g = rdf.Graph(fs, r, rdf.TAGS_FRAME)
    for bias, per_instance in ((100.0, 2), (-100.0, 1 + (2 ** (D + 1) - 1) + (2 ** (D + 1) - 2))):
        P["b_s"][0] = bias
        want, logs = oracle_run(P, tb, D)
        h, _ = g.eval_trees(rdf.Graph.device_trees(tb), rdf.Graph.device_params(P), rdf.F32, max_invocations=B * per_instance + 8)
        assert g.stats()["invocations"] == B * per_instance
        assert np.abs(h.cpu().numpy() - want).max() / np.abs(want).max() <= TOL


def test_topdown_is_forward_fp32_only():
    V, H, D, B = 50, 16, 3, 8
    P = workloads.topdown_params(7, V, H)
    tb = workloads.topdown_batch(7, B, V)
    fs, r = rdf.topdown_program(D)
    g = rdf.Graph(fs, r, rdf.TAGS_FRAME)
    dt, dp = rdf.Graph.device_trees(tb), rdf.Graph.device_params(P)
    with pytest.raises(rdf.RdfError) as e:
        g.eval_trees(dt, dp, rdf.BF16, max_invocations=4096)
    assert e.value.code == -11
    with pytest.raises(rdf.RdfError) as e:
        g.grad_trees(dt, dp, rdf.F32, max_invocations=4096)
    assert e.value.code == -11
    # an undersized frame table is a status code and the graph stays usable
    with pytest.raises(rdf.RdfError) as e:
        g.eval_trees(dt, dp, rdf.F32, max_invocations=B)
    assert e.value.code == -6
    want, _ = oracle_run(P, tb, D)
    h, _ = g.eval_trees(dt, dp, rdf.F32, max_invocations=4096)
    assert np.abs(h.cpu().numpy() - want).max() / np.abs(want).max() <= TOL


def test_topdown_full_size_as_benchmarked():
    """The workload `bench.py --workload 6` times (8192 seeds, H = 128, depth limit 10, frame table of 256 frames per
    seed): every instance against the oracle -- the root state of each decisive instance, the number of invocations
    of the whole batch when every instance is decisive, else of the decisive ones through the Call records."""
    cfg = workloads.config(6)
    tb, P, D = cfg["trees"], cfg["params"], cfg["D"]
    want, logs = oracle_run(P, tb, D)
    total = sum(1 + l["expand"] + l["child"] for l in logs)
    fs, r = rdf.topdown_program(D)
    g = rdf.Graph(fs, r, rdf.TAGS_FRAME)
    h, _ = g.eval_trees(rdf.Graph.device_trees(tb), rdf.Graph.device_params(P), rdf.F32, max_invocations=cfg["max_invocations"])
    h = h.cpu().numpy()
    st = g.stats()
    decisive = np.array([l["margin"] > MARGIN for l in logs])
    assert decisive.mean() >= 0.99, decisive.mean()
    err = np.abs(h[decisive] - want[decisive]).max() / np.abs(want[decisive]).max()
    assert err <= TOL, err
    # an instance that is not decisive may have grown another tree: the totals then differ by at most its size
    slack = sum(2 * (2 ** (D + 1)) for d in decisive if not d)
    assert abs(st["invocations"] - total) <= slack, (st["invocations"], total, slack)
