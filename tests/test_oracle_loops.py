"""Tagged iteration in the oracle (Section 2.3, Figure 1) and its composition with recursion (Section 5.1: loops and
function calls share the one tag stack).  Pins: the three semantic equations on bare nodes; the census of Figure 1;
closed forms of the loop programs; the tags the iterations run under (counter on top of the enclosing tag, inner
counter first for nested loops, a call's label on top of the counter); hiatons on or off give the same results."""
import pytest

from oracle import direct, programs, tagged, transform
from oracle.graphs import FunctionGraph


def _run(prog, x, dead=False):
    g = transform.transform(prog)
    return g, tagged.run(g, {0: x}, programs.INT_OPS, dead_tokens=dead, max_firings=2_000_000)


def test_enter_exit_next_equations():
    r = FunctionGraph("result", 1)
    e = r.enter(r.param(0))
    n1 = r.next_(e)
    n2 = r.next_(n1)
    r.output(r.exit_(n2))
    g = transform.transform([r])
    res = tagged.run(g, {0: 41}, programs.INT_OPS)
    assert res.enters == [(0,)]                      # Enter <t, d> = <0:t, d>
    assert res.nexts == [(1,), (2,)]                 # Next <n:t, d> = <(n+1):t, d>
    assert res.exits == [(2,)] and res.outputs == {(): 41}     # Exit <n:t, d> = <t, d>
    # nested: a second Enter puts its counter in front
    r = FunctionGraph("result", 1)
    a = r.next_(r.enter(r.param(0)))                 # [1]
    b = r.next_(r.next_(r.enter(a)))                 # [2, 1]
    r.output(r.exit_(r.exit_(b)))
    res = tagged.run(transform.transform([r]), {0: 7}, programs.INT_OPS)
    assert res.enters == [(0,), (0, 1)] and res.nexts == [(1,), (1, 1), (2, 1)] and res.exits == [(2, 1), (1,)]
    assert res.outputs == {(): 7}


def test_figure_1_structure():
    g = transform.transform(programs.sum_loop_program())
    # per loop-carried variable one Enter, one Merge fed by Enter and Next, one Switch, one Next; one Exit for the value
    assert g.count("Enter") == 3 and g.count("merge", "loop") == 3 and g.count("switch") == 3 and g.count("Next") == 3
    assert g.count("Exit") == 1
    for m in (n for n in g.nodes if n.kind == "merge"):
        kinds = sorted(g.nodes[e.src].kind for e in g.in_edges(m.id))
        assert kinds == ["Enter", "Next"]
    (ex,) = [n for n in g.nodes if n.kind == "Exit"]
    (e,) = g.in_edges(ex.id)
    assert g.nodes[e.src].kind == "switch" and e.src_port == 1          # the side taken when the condition fails
    for nx in (n for n in g.nodes if n.kind == "Next"):
        # what feeds Next comes from the true side of a Switch (through the body)
        seen, todo = set(), [nx.id]
        while todo:
            for e in g.in_edges(todo.pop()):
                if g.nodes[e.src].kind == "switch":
                    assert e.src_port == 0
                elif e.src not in seen:
                    seen.add(e.src)
                    todo.append(e.src)


@pytest.mark.parametrize("n", [0, 1, 2, 7, 40])
def test_sum_loop(n):
    _, res = _run(programs.sum_loop_program(), n)
    assert res.value == n * (n - 1) // 2 == direct.sum_to(n)
    assert res.enters == [(0,)] * 3                                     # the three variables enter under [0]
    assert sorted(set(res.nexts)) == [(k,) for k in range(1, n + 1)]    # iteration k runs under [k]
    assert res.exits == [(n,)]
    assert res.max_depth == 1
    _, dead = _run(programs.sum_loop_program(), n, dead=True)
    assert dead.value == res.value


@pytest.mark.parametrize("n", [0, 1, 2, 5, 9])
def test_nested_loops_tags(n):
    _, res = _run(programs.pairs_loop_program(), n)
    assert res.value == n * (n - 1) // 2 == direct.pairs(n)
    inner = {t for t in res.nexts if len(t) == 2}
    assert inner == {(j, i) for i in range(n) for j in range(1, i + 1)}          # [j, i]: inner counter first
    assert {t for t in res.nexts if len(t) == 1} == {(i,) for i in range(1, n + 1)}
    assert res.max_depth == (2 if n > 0 else 1)
    _, dead = _run(programs.pairs_loop_program(), n, dead=True)
    assert dead.value == res.value


@pytest.mark.parametrize("x", [0, 1, 2, 3, 10, 30, 97])
def test_function_called_from_a_loop_body(x):
    _, res = _run(programs.primes_loop_program(), x)
    assert res.value == direct.primes(x)
    # every invocation of isprime carries its label on top of the counter of the iteration that called it;
    # iteration k (k = 0, 1, ..) tests i = 2 + k
    top = {t for t in res.calls if len(t) == 2}
    assert top == {(0, k) for k in range(max(0, x - 1))}
    for t, a in res.calls.items():
        assert a[0] == 2 + t[-1]                                         # the number under test


@pytest.mark.parametrize("x", [0, 1, 2, 6, 12])
def test_loop_inside_a_recursive_function(x):
    _, res = _run(programs.tri_program(), x)
    assert res.value == (x - 1) * x * (x + 1) // 6 == direct.tri(x)      # sum of the triangular numbers below x
    # the loop of activation tri(m) runs under [k, 1, .., 1, 0]: counter on top of the activation's call labels
    depth = {}
    for t in res.nexts:
        depth.setdefault(t[1:], set()).add(t[0])
    want = {}
    for m in range(x, 0, -1):
        tag = (1,) * (x - m) + (0,)
        want[tag] = set(range(1, m + 1))
    assert depth == want
    _, dead = _run(programs.tri_program(), x, dead=True)
    assert dead.value == res.value
