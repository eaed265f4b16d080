"""rdf_eval_noalloc: evaluation for callers that cannot allocate device memory
(a host application that bans cudaMalloc after start-up, a pool that is already
fully handed out, a latency-critical path).  The entry point takes its scratch
from a 16 MiB array built into the library instead of a caller workspace.

Checked here, through the C boundary: its results equal those of rdf_eval
exactly (integer results: bit for bit) and those of the CPU oracle, on two calls
in a row with different inputs -- the second call must not see anything the first
one left in the shared array -- for an integer program and for a small TreeRNN,
and a batch that needs more than the built-in array is refused.
Collected last on purpose (file name), and self-contained so that it also passes
when run alone in a fresh process."""
import numpy as np
import pytest

import workloads
import paper_2410_20225_b200 as rdf
from oracle import direct
from paper_2410_20225_b200 import binding as bd

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def _calls(n):
    a, b = 0, 1
    for _ in range(n + 1):
        a, b = b, a + b
    return 2 * a - 1          # invocations of fib(n): 2 F(n+1) - 1


@pytest.mark.parametrize("mode", [rdf.TAGS_PATH, rdf.TAGS_FRAME])
def test_noalloc_matches_rdf_eval_twice_in_a_row(mode):
    fs, r = rdf.fib_program()
    g_ref = rdf.Graph(fs, r, mode)
    g = rdf.Graph(fs, r, mode)
    for seed in (11, 12):                                # two calls in a row, different inputs
        x_host = workloads.fib_batch(seed=seed, B=200, n_hi=12)
        n_inv = int(sum(_calls(int(n)) for n in x_host))
        x = torch.from_numpy(x_host).cuda()
        want, _ = g_ref.eval_int(x, max_invocations=n_inv)
        y = torch.full_like(x, -1)
        before = torch.cuda.memory_allocated()
        g.eval_int_noalloc(x, y, max_invocations=n_inv)
        assert torch.cuda.memory_allocated() == before   # nothing was taken from torch's allocator either
        assert torch.equal(y, want)
        assert y.tolist() == [direct.fib(int(n)) for n in x_host]        # and the recursive definition itself
        assert g.stats()["invocations"] == n_inv


def test_noalloc_tree_network_twice_in_a_row():
    """A small TreeRNN forward pass out of the built-in scratch: equal to rdf_eval bit for bit (the same kernels
    on the same inputs) and within the fp32 tolerance of the oracle, on two different batches in a row."""
    fs, r = rdf.tree_net_program("rnn")
    g_ref = rdf.Graph(fs, r, rdf.TAGS_FRAME)
    g = rdf.Graph(fs, r, rdf.TAGS_FRAME)
    for seed in (21, 22):
        cfg = workloads.config(3, seed=seed, B=32, V=200, H=32)
        tb = cfg["trees"]
        p = workloads.treernn_params(seed, 200, 32, 32)
        dt, dp = rdf.Graph.device_trees(tb), rdf.Graph.device_params(p)
        want, _ = g_ref.eval_trees(dt, dp)
        h = torch.full((tb.B, 32), float("nan"), dtype=torch.float32, device="cuda")
        before = torch.cuda.memory_allocated()
        g.eval_trees_noalloc(dt, dp, h)
        assert torch.cuda.memory_allocated() == before
        assert torch.equal(h, want)
        roots = direct.forward(tb, p, "rnn")
        assert float(np.abs(h.cpu().numpy() - roots).max() / np.abs(roots).max()) <= 1e-4
        assert g.stats()["invocations"] == tb.N


def test_noalloc_refuses_batches_beyond_the_builtin_scratch():
    fs, r = rdf.fib_program()
    g = rdf.Graph(fs, r, rdf.TAGS_PATH)
    x = torch.zeros(64, dtype=torch.int64, device="cuda")
    y = torch.full_like(x, -7)
    with pytest.raises(rdf.RdfError) as e:
        g.eval_int_noalloc(x, y, max_invocations=4_000_000)      # needs far more than 16 MiB of queues
    assert e.value.code == -3
    assert torch.all(y == -7)                                    # nothing was launched
    # and a fitting batch still works afterwards
    g.eval_int_noalloc(x, y, max_invocations=1000)
    assert torch.all(y == 0)
    assert bd.NOALLOC_SCRATCH_BYTES == 16 << 20
