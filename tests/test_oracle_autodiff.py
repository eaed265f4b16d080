"""Section 4 in the oracle: the gradient of the recursive tree networks as function graphs, transformed by the
algorithm of Section 3 and run by the literal tagged-token interpreter, in both forms the paper describes --
the naive one (a separate recursive gradient function that recomputes forward values) and the paired one
(call and gradient call under one label, forward values reaching the gradient operators by tag).
Pins: both give the gradients of the direct reverse recursion (itself pinned by finite differences and
autograd); in the paired run every tag carries a forward and a gradient argument and the tags are those of
the forward invocations; the paired run fires each forward operator once per tree node, the naive one more."""
import numpy as np
import pytest

import workloads
from oracle import autodiff, direct, tagged, transform


def _tiny(cell, seed=4, H=4, V=9):
    rng = np.random.default_rng(seed)
    shapes = [workloads.random_split_shape(rng, L) for L in (1, 2, 3, 5, 4)]
    tb = workloads.tree_batch_from_shapes(shapes, seed, vocab=V)
    p = (workloads.treernn_params if cell == "rnn" else workloads.treelstm_params)(seed, V, H, H)
    for k in p:
        if k.startswith("b"):
            p[k] = (0.2 * rng.standard_normal(p[k].shape)).astype(np.float32)
    return tb, p


def _run(program, tb, p, cell, counts=None):
    ops = autodiff.grad_ops(tb, p, cell)
    if counts is not None:
        for name in ("leaf", "cell", "cell_grad", "leaf_grad", "head_grad"):
            fn = ops[name]

            def counted(*a, _fn=fn, _name=name):
                counts[_name] = counts.get(_name, 0) + 1
                return _fn(*a)
            ops[name] = counted
    g = transform.transform(program)
    total, runs = None, []
    for t in range(tb.B):
        res = tagged.run(g, {0: int(tb.tree_root[t])}, ops, dead_tokens=False)
        G = res.value
        total = G if total is None else {k: total[k] + G[k] for k in G}
        runs.append(res)
    return g, total, runs


@pytest.mark.parametrize("cell", ["rnn", "lstm"])
def test_paired_equals_naive_equals_reverse_recursion(cell):
    tb, p = _tiny(cell)
    _, want, _ = direct.loss_and_grad(tb, p, cell)
    cn, cp = {}, {}
    _, Gn, _ = _run(autodiff.naive_grad_program(), tb, p, cell, cn)
    _, Gp, runs = _run(autodiff.paired_grad_program(), tb, p, cell, cp)
    for k in want:
        scale = max(np.abs(want[k]).max(), 1e-30)
        assert np.abs(Gn[k] - want[k]).max() / scale < 1e-12, k
        assert np.abs(Gp[k] - want[k]).max() / scale < 1e-12, k
    n_cells, n_leaves = tb.n_cells, tb.N - tb.n_cells
    # paired: nothing is recomputed -- one forward and one gradient firing per tree node
    assert cp == {"leaf": n_leaves, "cell": n_cells, "leaf_grad": n_leaves, "cell_grad": n_cells, "head_grad": tb.N}
    # naive: the gradient function recomputes forward values (every gradient invocation re-evaluates its
    # subtrees through calls of the forward function)
    assert cn["cell_grad"] == n_cells and cn["leaf_grad"] == n_leaves and cn["head_grad"] == tb.N
    assert cn["cell"] > n_cells and cn["leaf"] > n_leaves


def test_paired_invocations_share_the_tag_of_the_forward_call():
    tb, p = _tiny("rnn")
    _, _, runs = _run(autodiff.paired_grad_program(), tb, p, "rnn")
    for t, res in enumerate(runs):
        want = {tag: v for tag, v in direct.tree_invocations(tb, int(tb.tree_root[t]))}
        assert set(res.calls) == set(want)                         # the tags of the forward invocations, no others
        for tag, args in res.calls.items():
            assert set(args) == {0, 1}                             # forward argument and gradient argument, one tag
            assert args[0] == want[tag]
        # both outputs (state, parameter gradient) return under that tag too
        assert {k for k in res.returns_by_output} == {(tag, j) for tag in want for j in (0, 1)}


def test_gradient_graph_structure():
    """Census of the transformed graphs.  Paired: three call sites (one in `result`, two in the body), each with
    one Call_i per input (node, gradient) and one Return_i per output (state, parameter gradient); control edges
    connect the forward Call_i to the forward Return_i and the gradient Call_i to the gradient Return_i.
    Naive: the forward function is called from `result`, from its own body and from the gradient function."""
    g = transform.transform(autodiff.paired_grad_program())
    calls = [n for n in g.nodes if n.kind == "Call"]
    rets = [n for n in g.nodes if n.kind == "Return"]
    assert sorted((n.value, n.param) for n in calls) == [(i, k) for i in range(3) for k in range(2)]
    assert sorted((n.value, n.param) for n in rets) == [(i, j) for i in range(3) for j in range(2)]
    ctrl = [(g.nodes[e.src], g.nodes[e.dst]) for e in g.edges if e.control and g.nodes[e.src].kind == "Call"]
    assert sorted((a.value, a.param, b.value, b.param) for a, b in ctrl) == [(i, k, i, k) for i in range(3) for k in range(2)]
    assert g.count("merge", "entry") == 2 and g.count("fcall") == 0
    # every forward operator appears once: the gradient half reads its values, it holds no copy of it
    assert g.count("op", "cell") == 1 and g.count("op", "leaf") == 1
    n = transform.transform(autodiff.naive_grad_program())
    assert n.count("op", "cell") == 2 and n.count("op", "leaf") == 2       # the copies inside the gradient function
    by_callee = {}
    for c in (x for x in n.nodes if x.kind == "Call"):
        by_callee.setdefault(c.name, set()).add(c.value)
    assert by_callee == {"h": {0, 1, 2, 3, 4}, "h_grad": {0, 1, 2}}
