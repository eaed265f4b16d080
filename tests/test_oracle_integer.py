"""Pins for the integer side of the CPU oracle: the Section 3 transformation,
the Call/Return semantics and the tagged interpreter, against what the paper
and arithmetic fix (Figure 3, the factorial example, closed forms for fib)."""
import collections
import math
import os

import numpy as np
import pytest

import workloads
from oracle import direct, programs, tagged, transform
from oracle.graphs import FunctionGraph, Graph


# --------------------------------------------------------------------------
# Figure 3
# --------------------------------------------------------------------------
def _read_fig3(path):
    nodes, edges = {}, []
    for line in open(path):
        p = line.split()
        if not p or p[0].startswith("#"):
            continue
        if p[0] == "node":
            nodes[p[1]] = (p[2], p[3])
        elif p[0] == "edge":
            edges.append((p[1], int(p[2]), p[3], int(p[4]), False))
        elif p[0] == "control":
            edges.append((p[1], 0, p[2], -1, True))
    return nodes, edges


def _sig_fixture(kind, detail):
    return f"{kind}:{detail}"


def _sig_node(n):
    if n.kind == "op":
        return f"op:{n.name}"
    if n.kind in ("Call", "Return", "const"):
        return f"{n.kind}:{n.value}"
    if n.kind == "merge":
        return "merge:entry" if n.name == "entry" else "merge:if"
    return f"{n.kind}:-"


def test_transform_reproduces_figure_3(golden_dir):
    fn, fe = _read_fig3(os.path.join(golden_dir, "fact_fig3_graph.txt"))
    g = transform.transform(programs.fact_program())
    assert collections.Counter(_sig_fixture(*v) for v in fn.values()) == \
        collections.Counter(_sig_node(n) for n in g.nodes)
    want = collections.Counter((_sig_fixture(*fn[s]), sp, _sig_fixture(*fn[d]), dp, c) for s, sp, d, dp, c in fe)
    got = collections.Counter((_sig_node(g.nodes[e.src]), e.src_port if not e.control else 0,
                               _sig_node(g.nodes[e.dst]), e.dst_port, e.control) for e in g.edges)
    assert want == got
    # counts the text states: two Calls, two Returns, one control edge per pair
    assert g.count("Call") == 2 and g.count("Return") == 2 and g.count("merge") == 2 and g.count("switch") == 1
    assert g.count("fcall") == 0 and g.count("in") == 0 and g.count("out") == 1


def test_transform_general_counts():
    """n call sites of an m-parameter function give n*m Call nodes, n Return
    nodes, m entry Merges with n inputs each, n*m control edges (Section 3)."""
    r = FunctionGraph("result", 2)
    a = r.call("g", r.param(0), r.param(1))
    b = r.call("g", r.param(1), r.param(0))
    r.output(r.op("+", a, b))
    f = FunctionGraph("g", 2)
    x, y = f.param(0), f.param(1)
    t, e = f.switch(f.op("<", x, f.const(1)), x)
    rec = f.call("g", f.op("-", e, f.const(1)), y)
    f.output(f.merge(f.op("id", t), f.op("+", rec, f.const(1))))
    g = transform.transform([r, f])
    assert g.count("Call") == 3 * 2 and g.count("Return") == 3
    entry = [n for n in g.nodes if n.kind == "merge" and n.name == "entry"]
    assert len(entry) == 2 and all(n.n_in == 3 for n in entry)
    ctrl = [e for e in g.edges if e.control and g.nodes[e.src].kind == "Call"]
    assert len(ctrl) == 6
    assert all(g.nodes[e.dst].kind == "Return" and g.nodes[e.dst].value == g.nodes[e.src].value for e in ctrl)
    labels = sorted(n.value for n in g.nodes if n.kind == "Return")
    assert labels == [0, 1, 2]


# --------------------------------------------------------------------------
# Call_i / Return_i semantic equations
# --------------------------------------------------------------------------
def _single(kind, label):
    """in -> Call_label -> out, or in -> Return_label -> out, as a bare graph."""
    g = Graph()
    i = g.add("in", value=0)
    n = g.add(kind, value=label, n_in=1)
    o = g.add("out", n_in=1)
    g.connect(i, n, 0)
    g.connect(n, o, 0)
    return g


def test_call_prefixes_label():
    r = tagged.run(_single("Call", 7), {0: 42}, {})
    assert r.outputs == {(7,): 42}          # Call_i <t,d> = <i:t,d>


def test_call_then_return_is_identity_and_mismatch_is_silent():
    def chain(call_label, ret_label):
        g = Graph()
        i = g.add("in", value=0)
        c = g.add("Call", value=call_label, n_in=1)
        c2 = g.add("Call", value=3, n_in=1)
        r2 = g.add("Return", value=3, n_in=1)
        r = g.add("Return", value=ret_label, n_in=1)
        o = g.add("out", n_in=1)
        g.connect(i, c, 0)
        g.connect(c, c2, 0)
        g.connect(c2, r2, 0)
        g.connect(c2, r2, -1, control=True)
        g.connect(r2, r, 0)
        g.connect(c, r, -1, control=True)
        g.connect(r, o, 0)
        return g
    assert tagged.run(chain(5, 5), {0: -9}, {}).outputs == {(): -9}
    assert tagged.run(chain(5, 4), {0: -9}, {}).outputs == {}     # head 5 != 4: no output


def test_switch_merge_and_hiaton_propagation():
    f = FunctionGraph("result", 2)
    t, e = f.switch(f.param(0), f.param(1))
    f.output(f.merge(f.op("+", t, f.const(10)), f.op("*", e, f.const(3))))
    g = transform.transform([f])
    for dead in (True, False):
        assert tagged.run(g, {0: True, 1: 4}, programs.INT_OPS, dead_tokens=dead).value == 14
        assert tagged.run(g, {0: False, 1: 4}, programs.INT_OPS, dead_tokens=dead).value == 12
    assert tagged.run(g, {0: True, 1: 4}, programs.INT_OPS, dead_tokens=True).leftover == 0


# --------------------------------------------------------------------------
# the factorial example
# --------------------------------------------------------------------------
def test_fact_example_trace(golden_dir):
    inv, result = {}, None
    for line in open(os.path.join(golden_dir, "fact_trace.txt")):
        p = line.split()
        if p and p[0] == "invocation":
            inv[tuple(int(x) for x in p[1].split(","))] = (int(p[2]), int(p[3]))
        elif p and p[0] == "result":
            result = int(p[1])
    g = transform.transform(programs.fact_program())
    for dead in (True, False):
        r = tagged.run(g, {}, programs.INT_OPS, dead_tokens=dead)
        assert r.value == result == 11
        assert {t: (a[0], r.returns[t]) for t, a in r.calls.items()} == inv
    assert tagged.run(g, {}, programs.INT_OPS, dead_tokens=True).leftover == 0


@pytest.mark.parametrize("n", [1, 2, 5, 10, 15])
def test_fact_against_math_factorial(n):
    g = transform.transform(programs.fact_program(arg=n, addend=0))
    r = tagged.run(g, {}, programs.INT_OPS)
    assert r.value == math.factorial(n) == direct.fact(n)
    assert len(r.calls) == n and r.max_depth == n


# --------------------------------------------------------------------------
# fib: closed forms
# --------------------------------------------------------------------------
def _fib_iter(n):
    a, b = 0, 1
    for _ in range(n):
        a, b = b, a + b
    return a


def test_fib_values_recurrence_and_binet():
    phi = (1 + 5 ** 0.5) / 2
    for n in range(0, 26):
        assert direct.fib(n) == _fib_iter(n) == round(phi ** n / 5 ** 0.5)
    assert direct.fib(18) == 2584


@pytest.fixture(scope="module")
def fib_graph():
    return transform.transform(programs.fib_program())


def test_fib_graph_structure(fib_graph):
    g = fib_graph
    assert g.count("Call") == 3 and g.count("Return") == 3 and g.count("switch") == 1
    entry = [n for n in g.nodes if n.kind == "merge" and n.name == "entry"]
    assert len(entry) == 1 and entry[0].n_in == 3
    plus = [n for n in g.nodes if n.kind == "op" and n.name == "+"][0]
    srcs = sorted(g.nodes[e.src].value for e in g.in_edges(plus.id))
    assert srcs == [1, 2] and all(g.nodes[e.src].kind == "Return" for e in g.in_edges(plus.id))


@pytest.mark.parametrize("n", list(range(0, 13)) + [18])
def test_fib_tagged_equals_direct_and_counts(fib_graph, n):
    r = tagged.run(fib_graph, {0: n}, programs.INT_OPS)
    assert r.value == _fib_iter(n)
    assert r.leftover == 0
    # invocations: calls(n) = 2 F(n+1) - 1, tag depth max(1, n)
    assert len(r.calls) == 2 * _fib_iter(n + 1) - 1
    assert r.max_depth == max(1, n)
    # every invocation returns fib(argument); the trace equals direct recursion with call paths
    _, inv = direct.fib_invocations(n)
    assert {t: (a, v) for t, a, v in inv} == {t: (a[0], r.returns[t]) for t, a in r.calls.items()}
    for t, a in r.calls.items():
        assert r.returns[t] == _fib_iter(a[0])
    # tags: distinct by construction (dict keys), prefix closed, rooted at call site 0
    for t in r.calls:
        assert t[-1] == 0 and all(x in (1, 2) for x in t[:-1])
        assert len(t) == 1 or t[1:] in r.calls
    r2 = tagged.run(fib_graph, {0: n}, programs.INT_OPS, dead_tokens=False)
    assert r2.value == r.value and r2.calls == r.calls and r2.returns == r.returns


def test_fib_wave_widths_by_recurrence(fib_graph):
    """Invocations at tag depth d for n=18 follow w_n(d) = w_{n-1}(d-1) + w_{n-2}(d-1)."""
    def w(n, d):
        if d == 1:
            return 1
        if n < 2:
            return 0
        return w(n - 1, d - 1) + w(n - 2, d - 1)
    r = tagged.run(fib_graph, {0: 18}, programs.INT_OPS, dead_tokens=False)
    got = collections.Counter(len(t) for t in r.calls)
    assert [got[d] for d in range(1, 19)] == [w(18, d) for d in range(1, 19)]
    assert max(got.values()) == 2048 and got[13] == 2048
    assert sum(2 * _fib_iter(n + 1) - 1 for n in range(19)) == 21871


def test_fib_batch_totals():
    x = workloads.config(1)["x"]
    assert x.shape == (1024,) and x.min() >= 0 and x.max() <= 18
    total = sum(2 * _fib_iter(int(n) + 1) - 1 for n in x)
    assert abs(total - 1024 * 21871 / 19) < 0.1 * total      # the seed's N is near its expectation


# --------------------------------------------------------------------------
# integer tree folds pin the tree-walking machinery
# --------------------------------------------------------------------------
@pytest.fixture(scope="module")
def small_trees():
    return workloads.config(2, B=12)["trees"]


def test_tree_sum_count_height(small_trees):
    tb = small_trees
    ops = programs.tree_ops(tb)
    gsum = transform.transform(programs.tree_fold_program("tok", "+"))
    gcnt = transform.transform(programs.tree_fold_program("one", "+"))
    ghgt = transform.transform(programs.tree_fold_program("zero", "max", plus_one=True))
    sizes = tb.tree_sizes()
    for t in range(tb.B):
        root = int(tb.tree_root[t])
        sl = slice(root, root + int(sizes[t]))
        leaf_tok = tb.tok[sl][tb.left[sl] < 0]
        r = tagged.run(gsum, {0: root}, ops)
        assert r.value == int(leaf_tok.sum()) == direct.tree_fold(tb, root, lambda v: int(tb.tok[v]), lambda a, b: a + b)
        L = (sizes[t] + 1) // 2
        assert tagged.run(gcnt, {0: root}, ops).value == L
        assert len(r.calls) == 2 * L - 1                     # N = 2L - 1 invocations
        h = tagged.run(ghgt, {0: root}, ops).value
        assert h == direct.tree_fold(tb, root, lambda v: 0, lambda a, b: max(a, b) + 1)
        assert r.max_depth == h + 1
        # tag <-> tree node bijection: the tag is the reversed root-to-node path
        inv = direct.deep(direct.tree_invocations, tb, root)
        assert {tg: v for tg, v in inv} == {tg: a[0] for tg, a in r.calls.items()}


def test_chain_and_perfect_shapes():
    l, r = workloads.chain_tree_shape(40)
    tb = workloads.tree_batch_from_shapes([(l, r), workloads.perfect_tree_shape(5)], seed=1, vocab=10)
    height = lambda root: direct.deep(direct.tree_fold, tb, root, lambda v: 0, lambda a, b: max(a, b) + 1)  # noqa: E731
    assert height(int(tb.tree_root[0])) == 40 and height(int(tb.tree_root[1])) == 5
    assert tb.tree_sizes().tolist() == [81, 63]
    assert np.all(tb.right[tb.left >= 0] >= 0)
    # every right child of the chain is a leaf
    chain_int = [v for v in range(81) if tb.left[v] >= 0]
    assert all(tb.left[tb.right[v]] < 0 for v in chain_int)


# --------------------------------------------------------------------------
# multi-parameter and nested recursion (Table 1's ack and tak)
# --------------------------------------------------------------------------
def test_ackermann_closed_forms():
    """ack(1, n) = n + 2, ack(2, n) = 2n + 3, ack(3, n) = 2^(n+3) - 3."""
    for n in range(0, 7):
        assert direct.deep(direct.ack, 1, n) == n + 2
        assert direct.deep(direct.ack, 2, n) == 2 * n + 3
    for n in range(0, 5):
        assert direct.deep(direct.ack, 3, n) == 2 ** (n + 3) - 3


def test_takeuchi_known_values():
    """tak(x, y, z) with y >= x is z; tak(18, 12, 6) = 7 after 63 609 calls (the classic benchmark figures)."""
    assert direct.tak(3, 5, 9) == 9
    count = [0]
    assert direct.deep(direct.tak, 18, 12, 6, count) == 7 and count[0] == 63609


def test_transform_of_multi_parameter_functions():
    g = transform.transform(programs.tak_program())
    # 5 call sites of a 3-parameter function: 15 Call nodes, 5 Returns, 3 entry Merges with 5 inputs each
    assert g.count("Call") == 15 and g.count("Return") == 5
    entry = [n for n in g.nodes if n.kind == "merge" and n.name == "entry"]
    assert len(entry) == 3 and all(n.n_in == 5 for n in entry)
    ctrl = [e for e in g.edges if e.control and g.nodes[e.src].kind == "Call"]
    assert len(ctrl) == 15


@pytest.mark.parametrize("m,n", [(0, 3), (1, 2), (2, 0), (2, 3), (3, 2)])
def test_ack_tagged_equals_direct(m, n):
    g = transform.transform(programs.ack_program(m))
    count = [0]
    want = direct.deep(direct.ack, m, n, count)
    for dead in (True, False):
        r = tagged.run(g, {0: n}, programs.INT_OPS, dead_tokens=dead)
        assert r.value == want and len(r.calls) == count[0]
        # every invocation has both of its parameters, delivered by the two Call_i nodes of its call site
        assert all(sorted(a) == [0, 1] for a in r.calls.values())
        for tag, args in r.calls.items():
            assert r.returns[tag] == direct.deep(direct.ack, args[0], args[1])
    assert tagged.run(g, {0: n}, programs.INT_OPS, dead_tokens=True).leftover == 0


@pytest.mark.parametrize("x", [2, 5, 7, 9])
def test_tak_tagged_equals_direct(x):
    g = transform.transform(programs.tak_program(4, 2))
    count = [0]
    want = direct.tak(x, 4, 2, count)
    r = tagged.run(g, {0: x}, programs.INT_OPS, dead_tokens=False)
    assert r.value == want and len(r.calls) == count[0]
    for tag, args in r.calls.items():
        assert r.returns[tag] == direct.tak(args[0], args[1], args[2])


# ---------------------------------------------------------------------------
# primes: two mutually nested functions of two parameters, linear recursion
# ---------------------------------------------------------------------------
def _sieve_count(n):
    if n < 2:
        return 0
    mark = np.ones(n + 1, dtype=bool)
    mark[:2] = False
    for p in range(2, int(n ** 0.5) + 1):
        if mark[p]:
            mark[p * p::p] = False
    return int(mark.sum())


def test_primes_known_values():
    """pi(100) = 25, pi(1000) = 168, pi(10000) = 1229; 7919 is the 1000th prime."""
    assert [direct.primes(n) for n in (0, 1, 2, 3, 4, 100, 1000)] == [0, 0, 1, 2, 2, 25, 168]
    assert direct.primes(10000) == 1229
    assert direct.primes(7919) == 1000 and direct.primes(7918) == 999
    for n in (17, 289, 290, 2000, 7500):
        assert direct.primes(n) == _sieve_count(n)      # a sieve shares nothing with trial division


def test_remainder_operator():
    rem = programs.INT_OPS["%"]
    assert [rem(7, 3), rem(-7, 3), rem(7, -3), rem(-7, -3), rem(6, 3), rem(5, 0)] == [1, -1, 1, -1, 0, 0]
    assert rem(2 ** 62 + 5, 2 ** 31) == 5


@pytest.mark.parametrize("n", [0, 1, 2, 3, 10, 49, 120])
def test_primes_tagged_equals_direct(n):
    g = transform.transform(programs.primes_program())
    # 2 call sites of `count`, 2 of `isprime`, two parameters each
    assert g.count("Call") == 8 and g.count("Return") == 4
    count = [0]
    want = direct.primes(n, count)
    assert want == _sieve_count(n)
    for dead in (True, False):
        r = tagged.run(g, {0: n}, programs.INT_OPS, dead_tokens=dead)
        assert r.value == want and len(r.calls) == count[0]
        assert all(sorted(a) == [0, 1] for a in r.calls.values())
    r = tagged.run(g, {0: n}, programs.INT_OPS)
    assert r.leftover == 0
    # every invocation, as (arguments -> result): a `count(i, n)` returns pi(n) - pi(i - 1), an
    # `isprime(i, d)` whether i has no divisor in d .. sqrt(i); the two are told apart by the second
    # argument, which is n for count and at most sqrt(n) + 1 for isprime (n >= 5 makes them disjoint)
    if n >= 5:
        for tag, a in r.calls.items():
            if a[1] == n:
                assert r.returns[tag] == _sieve_count(n) - _sieve_count(a[0] - 1)
            else:
                no_divisor = all(a[0] % d for d in range(a[1], int(a[0] ** 0.5) + 1))
                assert r.returns[tag] == int(no_divisor)


def test_search_steered_by_a_call_result():
    """find(k) = k if T < fib(k) else find(k + 1): the Switch is driven by a callee's value.  Pinned by the iterative
    recurrence (the answer is the first index at or after k whose Fibonacci number exceeds T) and by the number of
    `find` invocations, answer - k + 1."""
    from oracle import transform, tagged
    for T in (0, 1, 50, 1000):
        fibs = [0, 1]
        while fibs[-1] <= T:
            fibs.append(fibs[-1] + fibs[-2])
        first = next(i for i, v in enumerate(fibs) if v > T)
        g = transform.transform(programs.find_program(T))
        for k in (0, 1, 3, first - 1, first, first + 2):
            if k < 0:
                continue
            want = max(k, first)
            count = {}
            assert direct.find_first_fib_above(k, T, count) == want and count["find"] == want - k + 1
            for dead in (True, False):
                r = tagged.run(g, {0: k}, programs.INT_OPS, dead_tokens=dead)
                assert r.value == want and (r.leftover == 0 or not dead)    # (without hiatons the constants of untaken sides stay parked)
