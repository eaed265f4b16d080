"""TEST INFRASTRUCTURE (CPU oracle) -- reverse-mode differentiation of the
recursive tree networks as *sets of function graphs*, in the two forms of
Section 4, for the literal tagged-token interpreter.

Section 4 gives every operator op_i a gradient operator op_i^grad that takes
the operator's original inputs and the gradients of its outputs and yields the
gradients of its inputs; forward values are retained.  For a user-defined
recursive function f it describes two ways to obtain f^grad:

  naive  (the set of graphs of the first figure of Section 4): differentiate
         the graph of f into a separate recursive function f^grad.  f^grad
         takes f's input and the output gradient, *recomputes* the forward
         values it needs (it contains copies of f's operators and calls f
         itself) and calls f^grad for the inner call.  result^grad calls f
         and then f^grad.

  paired (the transformed graph of the second figure): every invocation of f
         and its counterpart invocation of f^grad are replaced *together*, under
         the same label i, by one subgraph with n + m inputs (inputs of f,
         output gradients) and m + n outputs (outputs of f, input gradients).
         Forward operators and gradient operators of one invocation then carry
         the same tag, so the firing rule hands each gradient operator the
         forward values of its own invocation: nothing is recomputed.

Both are written here for the tree networks of the workloads,

    h(v) = leaf(tok v)                      if is_leaf(v)
         = cell(h(left v), h(right v))      otherwise,
    L    = sum over every node v of  -log softmax(W_s h(v) + b_s)[label v],

by applying that rule operator by operator: `leaf`, `cell` and the per-node
loss head each get their gradient operator; Switch is differentiated into a
Switch on the same predicate (the gradient goes down the branch that was
taken) and Merge into a Merge.  The node index v is an integer and has no
gradient; what a gradient function returns is the gradient with respect to
the *parameters* (E, W, b, W_s, b_s, ...), summed over the invocations below
it -- the usual fan-out rule (a reading: the paper does not discuss trainable
parameters inside a recursive body).

The gradient operators are plain numpy, fp64, each next to the formula it
implements.  A parameter gradient travels as a dict {name: array}.

Only tests, the smoke check and the CPU-baseline leg of the benchmark may
import anything under `oracle/`.
"""
from __future__ import annotations

import numpy as np

from .graphs import FunctionGraph
from .programs import sigmoid, tree_ops


# --------------------------------------------------------------------------
# operator tables: forward operators and their gradient operators
# --------------------------------------------------------------------------
def _zeros(P):
    return {k: np.zeros_like(v) for k, v in P.items()}


def _add(a, b):
    return {k: a[k] + b[k] for k in a}


def grad_ops(tb, params, cell: str):
    """Operators of the gradient programs.  A state is h (TreeRNN) or the pair
    (h, c) (TreeLSTM); a state gradient has the same shape as the state."""
    P = {k: np.asarray(v, dtype=np.float64) for k, v in params.items()}
    ops = tree_ops(tb)
    ops["fst"] = lambda t: t[0]
    ops["snd"] = lambda t: t[1]
    ops["third"] = lambda t: t[2]
    ops["padd"] = _add
    H = P["W_s"].shape[1]

    def head(h, v):
        z = P["W_s"] @ h + P["b_s"]
        p = np.exp(z) / np.exp(z).sum()
        p[int(tb.label[v])] -= 1.0          # softmax - onehot = dL_v / dz
        return p

    if cell == "rnn":
        ops["leaf"] = lambda tok: P["E"][tok]
        ops["cell"] = lambda a, b: np.tanh(P["W"] @ np.concatenate([a, b]) + P["b"])
        ops["zeros_like"] = lambda x: np.zeros_like(x)

        # loss head^grad: inputs (x, v, d) = the head's forward inputs and the gradient arriving at x from the
        # caller; outputs: total gradient at x, and the head's parameter gradients
        def head_grad(x, v, d):
            p = head(x, v)
            G = _zeros(P)
            G["W_s"] += np.outer(p, x)
            G["b_s"] += p
            return d + P["W_s"].T @ p, G

        # leaf^grad: inputs (tok, dx); the leaf is a row lookup, its gradient a row of dE
        def leaf_grad(tok, dx):
            G = _zeros(P)
            G["E"][tok] += dx
            return G

        # cell^grad: inputs (a, b, x, dx) with x = cell(a, b); outputs (da, db, parameter gradients)
        def cell_grad(a, b, x, dx):
            dz = dx * (1.0 - x * x)
            G = _zeros(P)
            G["W"] += np.outer(dz, np.concatenate([a, b]))
            G["b"] += dz
            dab = P["W"].T @ dz
            return dab[:H], dab[H:], G
    else:
        def leaf(tok):
            g = P["W_x"] @ P["E"][tok] + P["b_x"]
            c = sigmoid(g[:H]) * np.tanh(g[2 * H:])
            return sigmoid(g[H:2 * H]) * np.tanh(c), c

        def cell_fwd(a, b):
            (hl, cl), (hr, cr) = a, b
            g = P["W"] @ np.concatenate([hl, hr]) + P["b"]
            i, fl, fr, o = (sigmoid(g[k * H:(k + 1) * H]) for k in range(4))
            c = i * np.tanh(g[4 * H:]) + fl * cl + fr * cr
            return o * np.tanh(c), c

        ops["leaf"] = leaf
        ops["cell"] = cell_fwd
        ops["zeros_like"] = lambda s: (np.zeros_like(s[0]), np.zeros_like(s[1]))

        def head_grad(x, v, d):
            p = head(x[0], v)
            G = _zeros(P)
            G["W_s"] += np.outer(p, x[0])
            G["b_s"] += p
            return (d[0] + P["W_s"].T @ p, d[1]), G

        def leaf_grad(tok, dx):
            e = P["E"][tok]
            g = P["W_x"] @ e + P["b_x"]
            i, o, u = sigmoid(g[:H]), sigmoid(g[H:2 * H]), np.tanh(g[2 * H:])
            tc = np.tanh(i * u)
            dh, dc = dx
            dc = dc + dh * o * (1.0 - tc * tc)
            dg = np.concatenate([dc * u * i * (1 - i), dh * tc * o * (1 - o), dc * i * (1 - u * u)])
            G = _zeros(P)
            G["W_x"] += np.outer(dg, e)
            G["b_x"] += dg
            G["E"][tok] += P["W_x"].T @ dg
            return G

        def cell_grad(a, b, x, dx):
            (hl, cl), (hr, cr) = a, b
            xin = np.concatenate([hl, hr])
            g = P["W"] @ xin + P["b"]
            i, fl, fr, o = (sigmoid(g[k * H:(k + 1) * H]) for k in range(4))
            u = np.tanh(g[4 * H:])
            tc = np.tanh(x[1])
            dh, dc = dx
            dc = dc + dh * o * (1.0 - tc * tc)
            dg = np.concatenate([dc * u * i * (1 - i), dc * cl * fl * (1 - fl), dc * cr * fr * (1 - fr),
                                 dh * tc * o * (1 - o), dc * i * (1 - u * u)])
            G = _zeros(P)
            G["W"] += np.outer(dg, xin)
            G["b"] += dg
            dab = P["W"].T @ dg
            return (dab[:H], dc * fl), (dab[H:], dc * fr), G

    ops["head_grad"] = head_grad
    ops["leaf_grad"] = leaf_grad
    ops["cell_grad"] = cell_grad
    return ops


# --------------------------------------------------------------------------
# the forward function, shared by the naive set
# --------------------------------------------------------------------------
def _forward_function():
    f = FunctionGraph("h", 1)
    v = f.param(0)
    t, e = f.switch(f.op("is_leaf", v), v)
    a = f.call("h", f.op("left", e))
    b = f.call("h", f.op("right", e))
    f.output(f.merge(f.op("leaf", f.op("tok", t)), f.op("cell", a, b)))
    return f


def naive_grad_program():
    """{result, h, h_grad}: the gradient as a separate recursive function.

    result(root)   = h_grad(root, zeros_like(h(root)))        -- calls f, then f^grad
    h_grad(v, d)   = leaf:  x = leaf(tok v)                                   (forward value recomputed)
                            (dx, Gh) = head_grad(x, v, d);  Gh + leaf_grad(tok v, dx)
                     cell:  a = h(left v); b = h(right v); x = cell(a, b)     (forward values recomputed,
                            (dx, Gh) = head_grad(x, v, d)                      with calls of f itself)
                            (da, db, Gc) = cell_grad(a, b, x, dx)
                            Gh + Gc + h_grad(left v, da) + h_grad(right v, db)
    """
    r = FunctionGraph("result", 1)
    y = r.call("h", r.param(0))
    r.output(r.call("h_grad", r.param(0), r.op("zeros_like", y)))

    g = FunctionGraph("h_grad", 2)
    v, d = g.param(0), g.param(1)
    p = g.op("is_leaf", v)
    v_t, v_e = g.switch(p, v)
    d_t, d_e = g.switch(p, d)
    # leaf side
    tok = g.op("tok", v_t)
    x_t = g.op("leaf", tok)
    hg_t = g.op("head_grad", x_t, v_t, d_t)
    G_t = g.op("padd", g.op("snd", hg_t), g.op("leaf_grad", tok, g.op("fst", hg_t)))
    # cell side
    lv, rv = g.op("left", v_e), g.op("right", v_e)
    a, b = g.call("h", lv), g.call("h", rv)
    x_e = g.op("cell", a, b)
    hg_e = g.op("head_grad", x_e, v_e, d_e)
    cg = g.op("cell_grad", a, b, x_e, g.op("fst", hg_e))
    Gl = g.call("h_grad", lv, g.op("fst", cg))
    Gr = g.call("h_grad", rv, g.op("snd", cg))
    G_e = g.op("padd", g.op("padd", g.op("snd", hg_e), g.op("third", cg)), g.op("padd", Gl, Gr))
    g.output(g.merge(G_t, G_e))
    return [r, _forward_function(), g]


def paired_grad_program():
    """{result, hp}: one function hp(v, d) -> (state, G) that holds the forward operators and the gradient
    operators of an invocation; both of its call sites (and the one in `result`) pair the call of f with the
    call of f^grad under one label.  The gradient input of a call depends on that call's own forward output
    (through the caller's gradient operators), which is no cycle once the call node is replaced by its
    Call_i / Return_i nodes: the gradient Call_i simply fires later, under the same tag."""
    r = FunctionGraph("result", 1)
    c = r.call_open("hp", 2)
    r.set_arg(c, 0, r.param(0))
    r.set_arg(c, 1, r.op("zeros_like", (c, 0)))
    r.output((c, 1))

    f = FunctionGraph("hp", 2)
    f.grad_params, f.grad_outputs = {1}, {1}
    v, d = f.param(0), f.param(1)
    p = f.op("is_leaf", v)
    v_t, v_e = f.switch(p, v)
    d_t, d_e = f.switch(p, d)                 # the predicate waits under the invocation's tag until d arrives
    # leaf side
    tok = f.op("tok", v_t)
    x_t = f.op("leaf", tok)
    hg_t = f.op("head_grad", x_t, v_t, d_t)
    G_t = f.op("padd", f.op("snd", hg_t), f.op("leaf_grad", tok, f.op("fst", hg_t)))
    # cell side
    cl, cr = f.call_open("hp", 2), f.call_open("hp", 2)
    f.set_arg(cl, 0, f.op("left", v_e))
    f.set_arg(cr, 0, f.op("right", v_e))
    a, b = (cl, 0), (cr, 0)
    x_e = f.op("cell", a, b)
    hg_e = f.op("head_grad", x_e, v_e, d_e)
    cg = f.op("cell_grad", a, b, x_e, f.op("fst", hg_e))
    f.set_arg(cl, 1, f.op("fst", cg))
    f.set_arg(cr, 1, f.op("snd", cg))
    G_e = f.op("padd", f.op("padd", f.op("snd", hg_e), f.op("third", cg)), f.op("padd", (cl, 1), (cr, 1)))
    f.output(f.merge(x_t, x_e))
    f.output(f.merge(G_t, G_e))
    return [r, f]
