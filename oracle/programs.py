"""TEST INFRASTRUCTURE (CPU oracle) -- the source programs as sets of function
graphs (Figure 2 style) and the operator tables the interpreter needs.

Programs:
  * the factorial example of Section 2.4:  result = fact(3)+5;
    fact(n) = if (n==1) then n else n*fact(n-1);
  * fib(n) = if n<2 then n else fib(n-1)+fib(n-2).  The paper names `fib` in
    Table 1 without printing its definition; this is the textbook reading
    (fib 0 = 0, fib 1 = 1);
  * integer tree folds (sum of leaf tokens, leaf count, height) used to pin
    the tree-walking machinery;
  * the recursive tree networks: TreeRNN  h(v) = E[tok v] at a leaf,
    tanh(W [h(l); h(r)] + b) otherwise; the binary TreeLSTM; both optionally
    returning the pair (state, summed per-node loss).  The paper's Section 6.2
    names the TreeRNN sentiment model without giving its equations; the cell
    forms are the ones fixed by the workload list;
  * a top-down recursion whose Switch reads a vector value (`topdown_program`):
    the data-dependent recursion that Section 6.2's last paragraph points to.

Only tests, the smoke check and the CPU-baseline leg of the benchmark may
import anything under `oracle/`.
"""
from __future__ import annotations

import numpy as np

from .graphs import FunctionGraph


# --------------------------------------------------------------------------
# integer programs
# --------------------------------------------------------------------------
INT_OPS = {
    # unary operators with a built-in constant (inside a loop a constant is derived from a loop value, see
    # FunctionGraph.while_loop)
    "add1": lambda a: a + 1,
    "sub1": lambda a: a - 1,
    "zero": lambda a: 0,
    "two": lambda a: 2,
    "not": lambda a: not a,
    "+": lambda a, b: a + b,
    "-": lambda a, b: a - b,
    "*": lambda a, b: a * b,
    "<": lambda a, b: a < b,
    "==": lambda a, b: a == b,
    "id": lambda a: a,
    "max": lambda a, b: a if a > b else b,
    "one": lambda a: 1,
    # remainder of truncating division (sign of the dividend); 0 for a zero divisor
    "%": lambda a, b: 0 if b == 0 else (abs(a) % abs(b)) * (1 if a >= 0 else -1),
}


def fact_program(arg=3, addend=5):
    """Figure 2: the two graphs `result` and `fact`."""
    r = FunctionGraph("result", 0)
    r.output(r.op("+", r.const(addend), r.call("fact", r.const(arg))))
    f = FunctionGraph("fact", 1)
    n = f.param(0)
    t, e = f.switch(f.op("==", f.const(1), n), n)
    rec = f.call("fact", f.op("-", e, f.const(1)))
    f.output(f.merge(f.op("id", t), f.op("*", e, rec)))
    return [r, f]


def fib_program():
    r = FunctionGraph("result", 1)
    r.output(r.call("fib", r.param(0)))
    f = FunctionGraph("fib", 1)
    n = f.param(0)
    t, e = f.switch(f.op("<", n, f.const(2)), n)
    a = f.call("fib", f.op("-", e, f.const(1)))
    b = f.call("fib", f.op("-", e, f.const(2)))
    f.output(f.merge(f.op("id", t), f.op("+", a, b)))
    return [r, f]


def find_program(threshold=50):
    """Unbounded search steered by the result of a call:
        result(k) = find(k);   find(k) = k if threshold < fib(k) else find(k + 1)
    The Switch of `find` is driven by a value that a callee computed (the recursion cannot be unrolled into a loop with a
    known trip count: how far it goes is decided by fib)."""
    r = FunctionGraph("result", 1)
    r.output(r.call("find", r.param(0)))
    f = FunctionGraph("find", 1)
    k = f.param(0)
    p = f.op("<", f.const(threshold), f.call("fib", k))
    k_t, k_e = f.switch(p, k)
    f.output(f.merge(k_t, f.call("find", f.op("add1", k_e))))
    return [r, f, fib_program()[1]]


def ack_program(m_const=2):
    """result(x) = ack(m_const, x);
    ack(m, n) = if m == 0 then n + 1 else if n == 0 then ack(m - 1, 1) else ack(m - 1, ack(m, n - 1)).
    Table 1 names the Ackermann function without printing it: this is the textbook two-argument form.
    Every value a branch uses is routed through that branch's Switch (Figure 2), including the
    constant 1 of the second call, which is derived from the routed n ("one")."""
    r = FunctionGraph("result", 1)
    r.output(r.call("ack", r.const(m_const), r.param(0)))
    f = FunctionGraph("ack", 2)
    m, n = f.param(0), f.param(1)
    p1 = f.op("==", m, f.const(0))
    _, m_e = f.switch(p1, m)
    n_t, n_e = f.switch(p1, n)
    base = f.op("+", n_t, f.const(1))
    p2 = f.op("==", n_e, f.const(0))
    m_t2, m_e2 = f.switch(p2, m_e)
    n_t2, n_e2 = f.switch(p2, n_e)
    second = f.call("ack", f.op("-", m_t2, f.const(1)), f.op("one", n_t2))
    inner = f.call("ack", m_e2, f.op("-", n_e2, f.const(1)))
    third = f.call("ack", f.op("-", m_e2, f.const(1)), inner)
    f.output(f.merge(base, f.merge(second, third)))
    return [r, f]


def primes_program():
    """result(x) = count(2, x): how many primes are <= x, by trial division;
    count(i, n)   = if n < i then 0 else isprime(i, 2) + count(i + 1, n)
    isprime(i, d) = if i < d * d then 1 else if i % d == 0 then 0 else isprime(i, d + 1).
    Table 1 names `primes` without printing it: this is a textbook form that needs two functions of
    two parameters each, linear recursion as deep as x and a call next to another call's result.
    Constants used on one side of a conditional pass through that conditional's Switch."""
    r = FunctionGraph("result", 1)
    r.output(r.call("count", r.const(2), r.param(0)))
    c = FunctionGraph("count", 2)
    i, n = c.param(0), c.param(1)
    p = c.op("<", n, i)
    _, i_e = c.switch(p, i)
    _, n_e = c.switch(p, n)
    zero_t, _ = c.switch(p, c.const(0))
    _, two_e = c.switch(p, c.const(2))
    here = c.call("isprime", i_e, two_e)
    rest = c.call("count", c.op("+", i_e, c.const(1)), n_e)
    c.output(c.merge(c.op("id", zero_t), c.op("+", here, rest)))
    q = FunctionGraph("isprime", 2)
    i, d = q.param(0), q.param(1)
    p1 = q.op("<", i, q.op("*", d, d))
    _, i_e = q.switch(p1, i)
    _, d_e = q.switch(p1, d)
    one_t, _ = q.switch(p1, q.const(1))
    p2 = q.op("==", q.op("%", i_e, d_e), q.const(0))
    _, i_e2 = q.switch(p2, i_e)
    _, d_e2 = q.switch(p2, d_e)
    zero_t2, _ = q.switch(p2, q.const(0))
    again = q.call("isprime", i_e2, q.op("+", d_e2, q.const(1)))
    q.output(q.merge(q.op("id", one_t), q.merge(q.op("id", zero_t2), again)))
    return [r, c, q]


def tak_program(y_const=12, z_const=6):
    """result(x) = tak(x, y_const, z_const);
    tak(x, y, z) = if y < x then tak(tak(x-1, y, z), tak(y-1, z, x), tak(z-1, x, y)) else z.
    Table 1 names the Takeuchi function without printing it: this is the textbook form."""
    r = FunctionGraph("result", 1)
    r.output(r.call("tak", r.param(0), r.const(y_const), r.const(z_const)))
    f = FunctionGraph("tak", 3)
    x, y, z = f.param(0), f.param(1), f.param(2)
    p = f.op("<", y, x)
    x_t, _ = f.switch(p, x)
    y_t, _ = f.switch(p, y)
    z_t, z_e = f.switch(p, z)
    one = f.const(1)
    a = f.call("tak", f.op("-", x_t, one), y_t, z_t)
    b = f.call("tak", f.op("-", y_t, one), z_t, x_t)
    c = f.call("tak", f.op("-", z_t, one), x_t, y_t)
    f.output(f.merge(f.call("tak", a, b, c), f.op("id", z_e)))
    return [r, f]


# --------------------------------------------------------------------------
# tagged iteration (Section 2.3) alone, nested, with calls inside, and inside a recursive function
# --------------------------------------------------------------------------
def sum_loop_program():
    """result(n) = { s = 0; i = 0; while (i < n) { s = s + i; i = i + 1 }; s }  -- the while-loop of Figure 1 with the
    loop-carried variables (s, i, n)."""
    r = FunctionGraph("result", 1)
    n = r.param(0)
    out = r.while_loop([r.const(0), r.const(0), n],
                       lambda f, v: f.op("<", v[1], v[2]),
                       lambda f, v: [f.op("+", v[0], v[1]), f.op("add1", v[1]), f.op("id", v[2])], 0)
    r.output(out)
    return [r]


def pairs_loop_program():
    """result(n) = number of pairs (j, i) with 0 <= j < i < n, by two nested loops: the inner loop runs under tags
    [j, i] (inner counter first), as in the two-loop example of Section 2.3."""
    r = FunctionGraph("result", 1)
    n = r.param(0)

    def outer_body(f, v):                     # v = (acc, i, n)
        inner = f.while_loop([v[0], f.op("zero", v[1]), v[1]],          # (acc, j = 0, i)
                             lambda g, w: g.op("<", w[1], w[2]),
                             lambda g, w: [g.op("add1", w[0]), g.op("add1", w[1]), g.op("id", w[2])], 0)
        return [inner, f.op("add1", v[1]), f.op("id", v[2])]
    out = r.while_loop([r.const(0), r.const(0), n], lambda f, v: f.op("<", v[1], v[2]), outer_body, 0)
    r.output(out)
    return [r]


def primes_loop_program():
    """result(x) = { c = 0; i = 2; while (not x < i) { c = c + isprime(i, 2); i = i + 1 }; c } with the recursive
    isprime of `primes_program`: a function called from inside a loop body (the call's label goes on top of the
    iteration counter)."""
    r = FunctionGraph("result", 1)
    x = r.param(0)
    out = r.while_loop([r.const(0), r.const(2), x],
                       lambda f, v: f.op("not", f.op("<", v[2], v[1])),
                       lambda f, v: [f.op("+", v[0], f.call("isprime", v[1], f.op("two", v[1]))), f.op("add1", v[1]),
                                     f.op("id", v[2])], 0)
    r.output(out)
    q = [f for f in primes_program() if f.name == "isprime"][0]
    return [r, q]


def tri_program():
    """result(x) = tri(x);  tri(n) = if n < 1 then 0 else sumto(n) + tri(n - 1), where sumto(n) = 0 + 1 + .. + (n - 1)
    is a while-loop inside the body of the recursive function: loop frames on top of call frames."""
    r = FunctionGraph("result", 1)
    r.output(r.call("tri", r.param(0)))
    f = FunctionGraph("tri", 1)
    n = f.param(0)
    t, e = f.switch(f.op("<", n, f.const(1)), n)
    zero = f.op("zero", e)
    s = f.while_loop([zero, f.op("zero", e), e],
                     lambda g, v: g.op("<", v[1], v[2]),
                     lambda g, v: [g.op("+", v[0], v[1]), g.op("add1", v[1]), g.op("id", v[2])], 0)
    rec = f.call("tri", f.op("sub1", e))
    f.output(f.merge(f.op("zero", t), f.op("+", s, rec)))
    return [r, f]


def tree_fold_program(leaf_op: str, combine: str, plus_one: bool = False):
    """fold(v) = leaf_op(v) at a leaf, combine(fold(left v), fold(right v)) [+1]."""
    r = FunctionGraph("result", 1)
    r.output(r.call("fold", r.param(0)))
    f = FunctionGraph("fold", 1)
    v = f.param(0)
    t, e = f.switch(f.op("is_leaf", v), v)
    a = f.call("fold", f.op("left", e))
    b = f.call("fold", f.op("right", e))
    c = f.op(combine, a, b)
    if plus_one:
        c = f.op("+", c, f.const(1))
    f.output(f.merge(f.op(leaf_op, t), c))
    return [r, f]


def tree_ops(tb):
    """Accessors over one flat tree batch (indices are global node numbers)."""
    ops = dict(INT_OPS)
    ops.update({
        "is_leaf": lambda v: bool(tb.left[v] < 0),
        "left": lambda v: int(tb.left[v]),
        "right": lambda v: int(tb.right[v]),
        "tok": lambda v: int(tb.tok[v]),
        "one": lambda v: 1,
        "zero": lambda v: 0,
    })
    return ops


# --------------------------------------------------------------------------
# recursive tree networks
# --------------------------------------------------------------------------
def tree_net_program(cell: str, with_loss: bool):
    """h(v) = leaf(tok v) if is_leaf(v) else cell(h(left v), h(right v)).

    With `with_loss`, a call returns the pair (state, loss summed over the
    subtree) and `result` returns that pair for the root.
    cell is 'rnn' or 'lstm' (the operator names are cell_rnn/leaf_rnn etc.).
    """
    r = FunctionGraph("result", 1)
    r.output(r.call("h", r.param(0)))
    f = FunctionGraph("h", 1)
    v = f.param(0)
    t, e = f.switch(f.op("is_leaf", v), v)
    if not with_loss:
        leaf = f.op("leaf_" + cell, f.op("tok", t))
        a = f.call("h", f.op("left", e))
        b = f.call("h", f.op("right", e))
        f.output(f.merge(leaf, f.op("cell_" + cell, a, b)))
        return [r, f]
    leaf = f.op("leaf_" + cell, f.op("tok", t))
    leaf_pair = f.op("pack", leaf, f.op("node_loss", leaf, t))
    a = f.call("h", f.op("left", e))
    b = f.call("h", f.op("right", e))
    x = f.op("cell_" + cell, f.op("fst", a), f.op("fst", b))
    below = f.op("+", f.op("snd", a), f.op("snd", b))
    pair = f.op("pack", x, f.op("+", f.op("node_loss", x, e), below))
    f.output(f.merge(leaf_pair, pair))
    return [r, f]


def topdown_program():
    """The top-down recursion of `direct.topdown` as a set of function graphs:

        result(v)    = expand(seed(v), 0)          seed(v) = leaf_rnn(tok v)
        expand(h, d) = Merge( h,  cell_rnn(expand(left(h), d+1), expand(right(h), d+1)) )
                       with the Switches of h and d driven by  stop(h, d) = at_limit(d) or gate(h)
        left(h) = child_l(h)        right(h) = child_r(h)

    The predicate of the Switch reads the vector h: which Call nodes fire is decided by values computed during
    the run."""
    r = FunctionGraph("result", 1)
    r.output(r.call("expand", r.call("seed", r.param(0)), r.op("zero", r.param(0))))
    s = FunctionGraph("seed", 1)
    s.output(s.op("leaf_rnn", s.op("tok", s.param(0))))
    f = FunctionGraph("expand", 2)
    h, d = f.param(0), f.param(1)
    p = f.op("or", f.op("at_limit", d), f.op("gate", h))
    h_t, h_e = f.switch(p, h)
    _, d_e = f.switch(p, d)
    d1 = f.op("add1", d_e)
    a = f.call("expand", f.call("left", h_e), d1)
    b = f.call("expand", f.call("right", h_e), d1)
    f.output(f.merge(h_t, f.op("cell_rnn", a, b)))
    fl = FunctionGraph("left", 1)
    fl.output(fl.op("child_l", fl.param(0)))
    fr = FunctionGraph("right", 1)
    fr.output(fr.op("child_r", fr.param(0)))
    return [r, s, f, fl, fr]


def topdown_ops(tb, params, depth_limit):
    """Operator table for `topdown_program` (fp64)."""
    ops = tree_net_ops(tb, params, "rnn")
    P = {k: np.asarray(v, dtype=np.float64) for k, v in params.items()}
    H = P["W"].shape[0]
    ops["child_l"] = lambda h: np.tanh(P["W"][:, :H] @ h + P["b"])
    ops["child_r"] = lambda h: np.tanh(P["W"][:, H:] @ h + P["b"])
    ops["gate"] = lambda h: bool(P["W_s"][0] @ h + P["b_s"][0] > 0)
    ops["at_limit"] = lambda d: d >= depth_limit
    ops["or"] = lambda a, b: bool(a or b)
    return ops


def sigmoid(x):
    return 1.0 / (1.0 + np.exp(-x))


def node_loss_value(h, W_s, b_s, label):
    """-log softmax(W_s h + b_s)[label], written out directly."""
    z = W_s @ h + b_s
    p = np.exp(z) / np.exp(z).sum()
    return float(-np.log(p[label]))


def tree_net_ops(tb, params, cell: str):
    """Operator table for the tree networks; fp64 throughout.  An LSTM state
    is the pair (h, c); the loss head reads h."""
    P = {k: np.asarray(v, dtype=np.float64) for k, v in params.items()}
    ops = tree_ops(tb)
    ops["pack"] = lambda a, b: (a, b)
    ops["fst"] = lambda p: p[0]
    ops["snd"] = lambda p: p[1]
    if cell == "rnn":
        ops["leaf_rnn"] = lambda tok: P["E"][tok]
        ops["cell_rnn"] = lambda hl, hr: np.tanh(P["W"] @ np.concatenate([hl, hr]) + P["b"])
        ops["node_loss"] = lambda h, v: node_loss_value(h, P["W_s"], P["b_s"], int(tb.label[v]))
    else:
        H = P["W"].shape[0] // 5

        def leaf_lstm(tok):
            g = P["W_x"] @ P["E"][tok] + P["b_x"]
            i, o, u = g[:H], g[H:2 * H], g[2 * H:]
            c = sigmoid(i) * np.tanh(u)
            return (sigmoid(o) * np.tanh(c), c)

        def cell_lstm(l, r):
            (hl, cl), (hr, cr) = l, r
            g = P["W"] @ np.concatenate([hl, hr]) + P["b"]
            i, fl, fr, o, u = (g[k * H:(k + 1) * H] for k in range(5))
            c = sigmoid(i) * np.tanh(u) + sigmoid(fl) * cl + sigmoid(fr) * cr
            return (sigmoid(o) * np.tanh(c), c)

        ops["leaf_lstm"] = leaf_lstm
        ops["cell_lstm"] = cell_lstm
        ops["node_loss"] = lambda s, v: node_loss_value(s[0], P["W_s"], P["b_s"], int(tb.label[v]))
    return ops
