"""Host logic of the library, no GPU: the shared object loads and exports every
declared symbol; rdf_graph_build validates programs; the literal static graph it
produces (Section 3 transformation) is executed by the oracle's tagged-token
interpreter -- graph *data* crosses, no code -- and gives the oracle's results."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import workloads
import paper_2410_20225_b200 as rdf
from paper_2410_20225_b200 import binding as bd
from oracle import direct, programs, tagged, transform
from oracle.graphs import Graph as OGraph

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    lib = rdf.lib()
    header = open(os.path.join(ROOT, "include", "rdf.h")).read()
    declared = set(re.findall(r"^(?:int|void|const char\*)\s+(rdf_[a-z0-9_]+)\s*\(", header, flags=re.M))
    assert {"rdf_graph_build", "rdf_eval", "rdf_grad", "rdf_graph_free", "rdf_strerror"} <= declared
    for name in declared:
        assert hasattr(lib, name), name
    assert lib.rdf_strerror(-4).decode().startswith("call depth")
    assert set(bd.EXPORTS) <= declared


def test_struct_layouts_match_the_header():
    assert C.sizeof(bd.rdf_expr) == 24 and C.sizeof(bd.rdf_trace_rec) == 32 and bd.TRACE_DTYPE.itemsize == 32
    assert C.sizeof(bd.rdf_batch) == 10 * 8 and C.sizeof(bd.rdf_node) == 32 and C.sizeof(bd.rdf_edge) == 20
    assert C.sizeof(bd.rdf_params) == 6 * 4 + 7 * 8 and bd.rdf_params.E.offset == 24
    assert C.sizeof(bd.rdf_function) == 48 and bd.rdf_function.kind.offset == 28 and bd.rdf_function.next.offset == 36


# ----------------------------------------------------------------- errors
def _build(functions, result=0, mode=rdf.TAGS_PATH):
    return rdf.Graph(functions, result, mode)


def test_bad_programs_are_rejected():
    f = rdf.Function("result", 1)
    f.ret(f.call(5, f.param()))                       # unknown callee
    with pytest.raises(rdf.RdfError) as e:
        _build([f])
    assert e.value.code == -1
    fs, r = rdf.fib_program()
    fs[1].root = 99                                   # root out of range
    with pytest.raises(rdf.RdfError):
        _build(fs, r)
    fs, r = rdf.fib_program()
    with pytest.raises(rdf.RdfError):
        _build(fs, 7)                                 # no such `result`
    # a cycle among expressions
    g = rdf.Function("result", 1)
    g.exprs.append((bd.OP_ADD, 0, 0, -1, 0))
    g.root = 0
    with pytest.raises(rdf.RdfError):
        _build([g])
    # vector programs need frame tags
    fs, r = rdf.tree_net_program("rnn")
    with pytest.raises(rdf.RdfError) as e:
        _build(fs, r, rdf.TAGS_PATH)
    assert e.value.code == -11
    # several formal parameters live in the invocation's frame: packed path tags have no room for them
    a = rdf.Function("result", 1)
    a.ret(a.call(1, a.param(), a.const(3)))
    b = rdf.Function("g", 2)
    b.ret(b.param(1))
    with pytest.raises(rdf.RdfError) as e:
        _build([a, b], 0, rdf.TAGS_PATH)
    assert e.value.code == -11
    _build([a, b], 0, rdf.TAGS_FRAME)
    # a call site must give one argument per formal parameter
    a2 = rdf.Function("result", 1)
    a2.ret(a2.call(1, a2.param()))
    with pytest.raises(rdf.RdfError):
        _build([a2, b], 0, rdf.TAGS_FRAME)


def test_vector_programs_outside_the_executor_are_rejected():
    """An invocation owns one state slot, so its body may fire one vector operator, a cell reads the states
    of two callees, and integer operators, conditions and call arguments take integers.  Programs outside
    that are valid but not lowered: RDF_ERR_UNSUPPORTED at build time, not wrong states at run time."""
    def prog(body):
        r = rdf.Function("result", 1)
        r.ret(r.call(1, r.param()))
        f = rdf.Function("h", 1)
        v = f.param()
        f.ret(body(f, v))
        return [r, f]

    bad = [
        # a cell whose operand is another cell of the same invocation
        lambda f, v: f.if_(f.is_leaf(v), f.embed(f.tok(v)),
                           f.cell_rnn(f.cell_rnn(f.call(1, f.left(v)), f.call(1, f.right(v))), f.call(1, f.left(v)))),
        # a cell that reads an embedding computed in the same invocation
        lambda f, v: f.if_(f.is_leaf(v), f.embed(f.tok(v)), f.cell_rnn(f.embed(f.tok(v)), f.call(1, f.left(v)))),
        # an integer operator applied to a vector value
        lambda f, v: f.if_(f.is_leaf(v), f.embed(f.tok(v)), f.add(f.call(1, f.left(v)), f.const(1))),
        # a condition that is a vector value
        lambda f, v: f.if_(f.call(1, f.left(v)), f.embed(f.tok(v)), f.embed(f.tok(v))),
        # a vector value as a call argument
        lambda f, v: f.if_(f.is_leaf(v), f.embed(f.tok(v)), f.call(1, f.embed(f.tok(v)))),
        # the two sides of a conditional of different kinds
        lambda f, v: f.if_(f.is_leaf(v), f.embed(f.tok(v)), f.tok(v)),
    ]
    for body in bad:
        with pytest.raises(rdf.RdfError) as e:
            _build(prog(body), 0, rdf.TAGS_FRAME)
        assert e.value.code == -11
    # the supported shapes still build
    for cell in ("rnn", "lstm"):
        for with_loss in (False, True):
            fs, r = rdf.tree_net_program(cell, with_loss)
            _build(fs, r, rdf.TAGS_FRAME)


# ---------------------------------------- literal graph through the oracle
OPNAME = {bd.OP_ADD: "+", bd.OP_SUB: "-", bd.OP_MUL: "*", bd.OP_MAX: "max", bd.OP_REM: "%", bd.OP_LT: "<", bd.OP_EQ: "==",
          bd.OP_IS_LEAF: "is_leaf", bd.OP_LEFT: "left", bd.OP_RIGHT: "right", bd.OP_TOK: "tok",
          bd.OP_EMBED: "leaf_rnn", bd.OP_CELL_RNN: "cell_rnn", bd.OP_LEAF_LSTM: "leaf_lstm",
          bd.OP_CELL_LSTM: "cell_lstm", bd.OP_NODE_LOSS: "pass_state", bd.OP_CHILD_L: "child_l", bd.OP_CHILD_R: "child_r",
          bd.OP_GATE: "gate"}
KIND = {bd.NODE_IN: "in", bd.NODE_OUT: "out", bd.NODE_CONST: "const", bd.NODE_OP: "op", bd.NODE_SWITCH: "switch",
        bd.NODE_MERGE: "merge", bd.NODE_ENTRY_MERGE: "merge", bd.NODE_CALL: "Call", bd.NODE_RETURN: "Return",
        bd.NODE_ENTER: "Enter", bd.NODE_EXIT: "Exit", bd.NODE_NEXT: "Next"}


def _as_oracle_graph(desc):
    g = OGraph()
    for n in desc["nodes"]:
        kind = KIND[n["kind"]]
        value = n["value"]
        if kind in ("Call", "Return"):
            value = n["label"]
        elif kind == "in":
            value = n["param"]
        g.add(kind, name=OPNAME.get(n["op"], "entry" if n["kind"] == bd.NODE_ENTRY_MERGE else ""), value=value,
              func=str(n["func"]), n_in=n["n_in"], param=n["param"])
    for e in desc["edges"]:
        g.connect(e["src"], e["dst"], e["dst_port"], e["src_port"], bool(e["control"]))
    return g


def test_fact_graph_has_the_structure_of_figure_3():
    fs, r = rdf.fact_program()
    d = _build(fs, r).describe()
    kinds = [n["kind"] for n in d["nodes"]]
    assert kinds.count(bd.NODE_CALL) == 2 and kinds.count(bd.NODE_RETURN) == 2
    assert kinds.count(bd.NODE_ENTRY_MERGE) == 1 and kinds.count(bd.NODE_MERGE) == 1 and kinds.count(bd.NODE_SWITCH) == 1
    ctrl = [e for e in d["edges"] if e["control"]]
    call_ret = [e for e in ctrl if d["nodes"][e["src"]]["kind"] == bd.NODE_CALL]
    assert len(call_ret) == 2
    for e in call_ret:
        assert d["nodes"][e["dst"]]["kind"] == bd.NODE_RETURN
        assert d["nodes"][e["dst"]]["label"] == d["nodes"][e["src"]]["label"]
    assert len(ctrl) - len(call_ret) == 2          # entry Merge -> the two constants 1 (Figure 3)
    # Call_0 sits in `result`, Call_1 inside fact
    by_label = {n["label"]: n["func"] for n in d["nodes"] if n["kind"] == bd.NODE_CALL}
    assert by_label == {0: 0, 1: 1}
    # same node and edge census as the oracle's own transformation, up to the `id` node that
    # Figure 2 draws on the then-side
    og = transform.transform(programs.fact_program())
    assert len(d["nodes"]) == len(og.nodes) - 1 and len(d["edges"]) == len(og.edges) - 1
    g = _as_oracle_graph(d)
    for dead in (True, False):
        res = tagged.run(g, {}, programs.INT_OPS, dead_tokens=dead)
        assert res.value == 11
        assert {t: (a[0], res.returns[t]) for t, a in res.calls.items()} == \
            {(0,): (3, 6), (1, 0): (2, 2), (1, 1, 0): (1, 1)}


@pytest.mark.parametrize("n", [0, 1, 2, 7, 12])
def test_fib_literal_graph_runs_in_the_oracle(n):
    fs, r = rdf.fib_program()
    d = _build(fs, r).describe()
    assert d["n_labels"] == 3 and d["label_bits"] == 2 and d["n_match"] == 1
    res = tagged.run(_as_oracle_graph(d), {0: n}, programs.INT_OPS)
    og = tagged.run(transform.transform(programs.fib_program()), {0: n}, programs.INT_OPS)
    assert res.value == og.value == direct.fib(n)
    assert res.calls == og.calls and res.returns == og.returns and res.leftover == 0


@pytest.mark.parametrize("name,arg", [("ack", 0), ("ack", 3), ("tak", 3), ("tak", 9), ("primes", 1), ("primes", 30)])
def test_multi_parameter_literal_graphs_run_in_the_oracle(name, arg):
    """One Call_i node per formal parameter and one Return_i per call site; calls nested in arguments."""
    if name == "ack":
        (fs, r), oprog, want = rdf.ack_program(2), programs.ack_program(2), direct.ack(2, arg)
    elif name == "tak":
        (fs, r), oprog, want = rdf.tak_program(6, 2), programs.tak_program(6, 2), direct.tak(arg, 6, 2)
    else:
        (fs, r), oprog, want = rdf.primes_program(), programs.primes_program(), direct.primes(arg)
    d = _build(fs, r, rdf.TAGS_FRAME).describe()
    n_par = 3 if name == "tak" else 2
    sites = d["n_labels"]
    # per callee, the local call-site numbers are 0 .. (sites of that callee) - 1, `result`'s site first
    by_callee = {}
    for callee, local in zip(d["label_callee"], d["label_local"]):
        by_callee.setdefault(callee, []).append(local)
    assert all(sorted(v) == list(range(len(v))) for v in by_callee.values()) and d["label_local"][0] == 0
    kinds = [n["kind"] for n in d["nodes"]]
    assert kinds.count(bd.NODE_RETURN) == sites and kinds.count(bd.NODE_CALL) == sites * n_par
    res = tagged.run(_as_oracle_graph(d), {0: arg}, programs.INT_OPS)
    og = tagged.run(transform.transform(oprog), {0: arg}, programs.INT_OPS)
    assert res.value == og.value == want
    assert res.calls == og.calls and res.returns == og.returns and res.leftover == 0


def test_tree_literal_graphs_run_in_the_oracle():
    tb = workloads.config(2, B=6)["trees"]
    ops = programs.tree_ops(tb)
    for kind in ("sum", "count", "height"):
        fs, r = rdf.tree_fold_program(kind)
        g = _as_oracle_graph(_build(fs, r, rdf.TAGS_FRAME).describe())
        for t in range(tb.B):
            root = int(tb.tree_root[t])
            want = {"sum": lambda: direct.tree_fold(tb, root, lambda v: int(tb.tok[v]), lambda a, b: a + b),
                    "count": lambda: direct.tree_fold(tb, root, lambda v: 1, lambda a, b: a + b),
                    "height": lambda: direct.tree_fold(tb, root, lambda v: 0, lambda a, b: max(a, b) + 1)}[kind]()
            for dead in (True, False):
                assert tagged.run(g, {0: root}, ops, dead_tokens=dead).value == want


@pytest.mark.parametrize("cell", ["rnn", "lstm"])
def test_tree_net_literal_graph_runs_in_the_oracle(cell):
    rng = np.random.default_rng(0)
    tb = workloads.tree_batch_from_shapes([workloads.random_split_shape(rng, L) for L in (1, 2, 5, 7)], 3, vocab=9)
    p = (workloads.treernn_params if cell == "rnn" else workloads.treelstm_params)(3, 9, 4, 4)
    ops = programs.tree_net_ops(tb, p, cell)
    ops["pass_state"] = lambda s, v: s
    fs, r = rdf.tree_net_program(cell, with_loss=True)
    g = _as_oracle_graph(_build(fs, r, rdf.TAGS_FRAME).describe())
    want = direct.forward(tb, p, cell)
    for t in range(tb.B):
        res = tagged.run(g, {0: int(tb.tree_root[t])}, ops)
        got = res.value if cell == "rnn" else res.value[0]
        np.testing.assert_allclose(got, want[t], atol=1e-13)
        assert len(res.calls) == tb.tree_sizes()[t]


def test_condition_that_waits_for_a_call_literal_graph_runs_in_the_oracle():
    fs, r = rdf.find_program(50)
    g = _as_oracle_graph(_build(fs, r, rdf.TAGS_FRAME).describe())
    for k in (0, 4, 9, 10, 13):
        res = tagged.run(g, {0: k}, programs.INT_OPS)
        assert res.value == direct.find_first_fib_above(k, 50) and res.leftover == 0
    with pytest.raises(rdf.RdfError) as e:            # the parameter is read back from the frame after the call: frame tags
        _build(fs, r, rdf.TAGS_PATH)
    assert e.value.code == -11


def test_topdown_literal_graph_runs_in_the_oracle():
    """Recursion shaped by vector values (Section 6.2, last paragraph): the graph rdf_graph_build makes of the
    top-down program -- a Switch whose predicate comes from RDF_OP_GATE on a state -- run by the oracle's interpreter
    against the direct recursion."""
    V, H, D = 40, 6, 5
    P = workloads.topdown_params(5, V, H)
    tb = workloads.topdown_batch(5, 10, V)
    ops = programs.topdown_ops(tb, P, D)
    fs, r = rdf.topdown_program(D)
    desc = _build(fs, r, rdf.TAGS_FRAME).describe()
    g = _as_oracle_graph(desc)
    kinds = [n["kind"] for n in desc["nodes"]]
    # call sites: seed 1, expand 3 (one in result, two in expand), left 1, right 1; one Call_i per parameter
    assert kinds.count(bd.NODE_CALL) == 1 + 3 * 2 + 1 + 1 and kinds.count(bd.NODE_RETURN) == 6
    sizes = set()
    for b in range(tb.B):
        log = {}
        want = direct.topdown(P, int(tb.tok[b]), D, log)
        res = tagged.run(g, {0: int(tb.tree_root[b])}, ops)
        np.testing.assert_allclose(res.value, want, atol=1e-13)
        assert res.leftover == 0
        sizes.add(log["expand"])
    assert len(sizes) >= 3


def test_topdown_programs_outside_the_executor_are_rejected():
    def prog(expand_body, left_body=None, mode=rdf.TAGS_FRAME):
        r = rdf.Function("result", 1)
        r.ret(r.call(2, r.call(1, r.param()), r.const(0)))
        s = rdf.Function("seed", 1)
        s.ret(s.embed(s.tok(s.param())))
        f = rdf.Function("expand", 2)
        f.ret(expand_body(f, f.param(0), f.param(1)))
        fl = rdf.Function("left", 1)
        fl.ret((left_body or (lambda g, h: g.child_l(h)))(fl, fl.param()))
        return [r, s, f, fl], mode

    ok = lambda f, h, d: f.if_(f.max(f.lt(f.const(3), d), f.gate(h)), h,                      # noqa: E731
                               f.cell_rnn(f.call(2, f.call(3, h), f.add(d, f.const(1))), f.call(2, f.call(3, h), f.add(d, f.const(1)))))
    fs, mode = prog(ok)
    _build(fs, 0, mode)
    bad = [
        prog(ok, mode=rdf.TAGS_PATH),                                                          # states live in frames
        prog(lambda f, h, d: f.if_(f.gate(d), h, h)),                                          # a gate on an integer
        prog(lambda f, h, d: f.if_(f.gate(h), h, f.child_l(f.call(3, h)))),                    # a child operator on a call's result
        # two vector operators in one invocation (the child states computed where the cell is)
        prog(lambda f, h, d: f.if_(f.gate(h), h, f.cell_rnn(f.call(2, f.child_l(h), d), f.call(2, f.child_r(h), d)))),
        prog(ok, left_body=lambda g, h: g.child_l(g.child_r(h))),                              # a child operator on a computed state
        prog(lambda f, h, d: f.if_(f.gate(h), h, f.call(2, d, d))),                            # an integer where the callee takes a state
    ]
    for fs, mode in bad:
        with pytest.raises(rdf.RdfError) as e:
            _build(fs, 0, mode)
        assert e.value.code == -11


LOOPS = {"sum": (rdf.sum_loop_program, programs.sum_loop_program, direct.sum_to, [0, 1, 5, 17]),
         "pairs": (rdf.pairs_loop_program, programs.pairs_loop_program, direct.pairs, [0, 1, 4, 7]),
         "primes": (rdf.primes_loop_program, programs.primes_loop_program, direct.primes, [0, 2, 3, 20]),
         "tri": (rdf.tri_program, programs.tri_program, direct.tri, [0, 1, 3, 6])}


@pytest.mark.parametrize("name", sorted(LOOPS))
def test_loop_literal_graphs_run_in_the_oracle(name):
    """The literal graph the library builds for a loop (Figure 1 in place of the call of the loop definition) is run
    by the oracle's interpreter: the values of the plain definitions, and the same iteration and call tags as the
    oracle's own graph of the program."""
    make, oracle_prog, plain, xs = LOOPS[name]
    fs, r = make()
    d = _build(fs, r, rdf.TAGS_FRAME).describe()
    kinds = [n["kind"] for n in d["nodes"]]
    assert kinds.count(bd.NODE_ENTER) == kinds.count(bd.NODE_NEXT) and kinds.count(bd.NODE_ENTER) % 3 == 0
    assert kinds.count(bd.NODE_EXIT) == kinds.count(bd.NODE_ENTER) // 3                 # three variables per loop, one value
    g = _as_oracle_graph(d)
    og = transform.transform(oracle_prog())
    assert g.count("Enter") == og.count("Enter") and g.count("Next") == og.count("Next") and g.count("Exit") == og.count("Exit")
    assert g.count("Call") == og.count("Call") and g.count("Return") == og.count("Return")
    for x in xs:
        res = tagged.run(g, {0: x}, programs.INT_OPS, dead_tokens=False, max_firings=500000)
        want = tagged.run(og, {0: x}, programs.INT_OPS, dead_tokens=False, max_firings=500000)
        assert res.value == want.value == plain(x)
        assert sorted(res.nexts) == sorted(want.nexts) and sorted(res.enters) == sorted(want.enters)
        assert sorted(res.exits) == sorted(want.exits)
        assert {t: tuple(a[k] for k in sorted(a)) for t, a in res.calls.items()} == \
            {t: tuple(a[k] for k in sorted(a)) for t, a in want.calls.items()}


def test_bad_loops_are_rejected():
    fs, r = rdf.sum_loop_program()
    with pytest.raises(rdf.RdfError) as e:
        _build(fs, r, rdf.TAGS_PATH)                       # the iteration counter lives beside a frame id
    assert e.value.code == -11
    fs, r = rdf.sum_loop_program()
    fs[1].cond = 99
    with pytest.raises(rdf.RdfError):
        _build(fs, r, rdf.TAGS_FRAME)
    # a call in the condition is not lowered
    fs, r = rdf.primes_loop_program()
    lp = fs[1]
    lp.cond = lp.call(2, lp.param(1), lp.const(2))
    with pytest.raises(rdf.RdfError) as e:
        _build(fs, r, rdf.TAGS_FRAME)
    assert e.value.code == -11
    # a loop that contains itself has no finite graph
    a = rdf.Function("result", 1)
    a.ret(a.call(1, a.param()))
    lp = rdf.Function("self", 1)
    v = lp.param()
    lp.loop(lp.lt(v, lp.const(3)), [lp.call(1, v)], v)
    with pytest.raises(rdf.RdfError):
        _build([a, lp], 0, rdf.TAGS_FRAME)


def test_product_path_has_no_cpu_route():
    """Without a CUDA device the evaluation entry points refuse to run."""
    import torch
    if torch.cuda.is_available():
        pytest.skip("GPU present")
    fs, r = rdf.fib_program()
    g = _build(fs, r)
    with pytest.raises(RuntimeError):
        g.eval_int(torch.zeros(4, dtype=torch.int64), 100)
    for name in ("binding.py", "__init__.py", "build.py"):
        src = open(os.path.join(ROOT, "paper_2410_20225_b200", name)).read()
        assert "import oracle" not in src and "from oracle" not in src
