"""TEST INFRASTRUCTURE (CPU oracle) -- direct recursive evaluation.

The transformed graph computes exactly what the recursive definitions say
(Section 3: one can run the resulting graph and verify that it computes the
desired output), so the definition of a correct result is plain recursion.
This module is that definition written out in Python/numpy (fp64), plus the
reverse-mode gradient written as the reverse recursion (Section 4: for each
operator a gradient operator that takes the original inputs and the output
gradients; forward values are retained).  Parameter gradients are summed over
every invocation that read the parameter (the usual fan-out rule; the paper
does not discuss trainable parameters inside a recursive body).

`fib_invocations` and `tree_invocations` additionally carry the list of call-site labels, which is
the tag the invocation has in the tagged execution (Call_i prefixes i).

Nothing here is blocked, fused or reordered; recursion depth is handled by
running in a thread with a large stack.

Only tests, the smoke check and the CPU-baseline leg of the benchmark may
import anything under `oracle/`.
"""
from __future__ import annotations

import sys
import threading

import numpy as np


def deep(fn, *args, **kw):
    """Run fn(*args) in a thread whose stack admits recursion depth ~1e5."""
    out = {}

    def target():
        try:
            out["v"] = fn(*args, **kw)
        except BaseException as e:  # re-raised in the caller
            out["e"] = e

    old = sys.getrecursionlimit()
    sys.setrecursionlimit(max(old, 200000))
    threading.stack_size(1024 * 1024 * 1024)
    t = threading.Thread(target=target)
    t.start()
    t.join()
    threading.stack_size(0)
    sys.setrecursionlimit(old)
    if "e" in out:
        raise out["e"]
    return out["v"]


# --------------------------------------------------------------------------
# integers
# --------------------------------------------------------------------------
def fact(n):
    return n if n == 1 else n * fact(n - 1)


def fib(n):
    return n if n < 2 else fib(n - 1) + fib(n - 2)


def ack(m, n, count=None):
    """Textbook Ackermann function; `count` (a one-element list) counts the invocations."""
    if count is not None:
        count[0] += 1
    if m == 0:
        return n + 1
    if n == 0:
        return ack(m - 1, 1, count)
    return ack(m - 1, ack(m, n - 1, count), count)


def tak(x, y, z, count=None):
    """Textbook Takeuchi function."""
    if count is not None:
        count[0] += 1
    if y < x:
        return tak(tak(x - 1, y, z, count), tak(y - 1, z, x, count), tak(z - 1, x, y, count), count)
    return z


def primes(n, count=None):
    """How many primes are <= n: every i in 2..n is tried against d = 2, 3, ... while d * d <= i.
    `count` (a one-element list) receives the number of invocations the recursive definition
    count/isprime makes: one `count` per i in 2..n+1 and one `isprime` per divisor tried."""
    found = 0
    calls = 0
    for i in range(2, n + 1):
        d = 2
        calls += 1
        while d * d <= i and i % d != 0:
            d += 1
            calls += 1
        if d * d > i:
            found += 1
    if count is not None:
        count[0] += calls + max(n, 1)      # count(2..n+1, n): n invocations (one when n < 2)
    return found


def find_first_fib_above(k, threshold, count=None):
    """find(k) = k if threshold < fib(k) else find(k + 1), written as the recursion it is; `count`, if a dict, receives
    the number of `find` invocations."""
    if count is not None:
        count["find"] = count.get("find", 0) + 1
    return k if threshold < fib(k) else find_first_fib_above(k + 1, threshold, count)


def sum_to(n):
    """0 + 1 + .. + (n - 1), by the loop itself."""
    s, i = 0, 0
    while i < n:
        s, i = s + i, i + 1
    return s


def pairs(n):
    """Number of pairs (j, i) with 0 <= j < i < n, by the two nested loops."""
    acc, i = 0, 0
    while i < n:
        j = 0
        while j < i:
            acc, j = acc + 1, j + 1
        i += 1
    return acc


def tri(n):
    """tri(n) = 0 if n < 1 else sum_to(n) + tri(n - 1)."""
    return 0 if n < 1 else sum_to(n) + tri(n - 1)


def fib_invocations(n, tag=(0,), out=None):
    """Every invocation of fib below the call `result = fib(n)` as
    (tag, argument, result); the call in `result` is call site 0, the two
    calls in the body are sites 1 and 2; a tag lists sites innermost first."""
    if out is None:
        out = []
    if n < 2:
        r = n
    else:
        r = fib_invocations(n - 1, (1,) + tag, out)[0] + fib_invocations(n - 2, (2,) + tag, out)[0]
    out.append((tag, n, r))
    return r, out


def tree_fold(tb, v, leaf_fn, combine):
    if tb.left[v] < 0:
        return leaf_fn(v)
    return combine(tree_fold(tb, int(tb.left[v]), leaf_fn, combine),
                   tree_fold(tb, int(tb.right[v]), leaf_fn, combine))


def tree_invocations(tb, v, tag=(0,), out=None):
    """(tag, node) for every invocation of a binary tree recursion rooted at v
    (call sites: 0 in `result`, 1 = left child, 2 = right child)."""
    if out is None:
        out = []
    out.append((tag, v))
    if tb.left[v] >= 0:
        tree_invocations(tb, int(tb.left[v]), (1,) + tag, out)
        tree_invocations(tb, int(tb.right[v]), (2,) + tag, out)
    return out


# --------------------------------------------------------------------------
# tree networks, forward
# --------------------------------------------------------------------------
def _f64(params):
    return {k: np.asarray(v, dtype=np.float64) for k, v in params.items()}


def sigmoid(x):
    return 1.0 / (1.0 + np.exp(-x))


def rnn_cell(P, hl, hr):
    """tanh(W [h_l; h_r] + b)"""
    return np.tanh(P["W"] @ np.concatenate([hl, hr]) + P["b"])


def lstm_leaf(P, e):
    """[i; o; u] = W_x e + b_x;  c = s(i) tanh(u);  h = s(o) tanh(c)"""
    H = P["W_x"].shape[0] // 3
    g = P["W_x"] @ e + P["b_x"]
    c = sigmoid(g[:H]) * np.tanh(g[2 * H:])
    return sigmoid(g[H:2 * H]) * np.tanh(c), c


def lstm_cell(P, hl, cl, hr, cr):
    """[i; f_l; f_r; o; u] = W [h_l; h_r] + b;
    c = s(i) tanh(u) + s(f_l) c_l + s(f_r) c_r;  h = s(o) tanh(c)"""
    H = P["W"].shape[0] // 5
    g = P["W"] @ np.concatenate([hl, hr]) + P["b"]
    i, fl, fr, o, u = (g[k * H:(k + 1) * H] for k in range(5))
    c = sigmoid(i) * np.tanh(u) + sigmoid(fl) * cl + sigmoid(fr) * cr
    return sigmoid(o) * np.tanh(c), c


def treernn_h(tb, P, v, store=None):
    """h(v) = E[tok v] at a leaf, cell(h(left v), h(right v)) otherwise."""
    if tb.left[v] < 0:
        h = P["E"][tb.tok[v]]
    else:
        hl = treernn_h(tb, P, int(tb.left[v]), store)
        hr = treernn_h(tb, P, int(tb.right[v]), store)
        h = rnn_cell(P, hl, hr)
    if store is not None:
        store[v] = h
    return h


def treelstm_hc(tb, P, v, store=None):
    """Binary TreeLSTM state (h, c) of node v (bottom-up; a leaf has no child
    cell state, hence no forget gates)."""
    if tb.left[v] < 0:
        h, c = lstm_leaf(P, P["E"][tb.tok[v]])
    else:
        hl, cl = treelstm_hc(tb, P, int(tb.left[v]), store)
        hr, cr = treelstm_hc(tb, P, int(tb.right[v]), store)
        h, c = lstm_cell(P, hl, cl, hr, cr)
    if store is not None:
        store[v] = (h, c)
    return h, c


def topdown(params, tok, depth_limit, log=None):
    """Recursion whose *shape* depends on the values it computes -- the kind of definition Section 6.2 closes
    with (a tree generated top-down by the model cannot be written as an iteration over a given structure):

        result(tok)  = expand(E[tok], 0)
        expand(h, d) = h                                                 if d >= D or gate(h)
                     = cell(expand(left(h), d+1), expand(right(h), d+1))   otherwise
        left(h)  = tanh(W[:, :H] h + b)      right(h) = tanh(W[:, H:] h + b)
        gate(h)  = W_s[0] . h + b_s[0] > 0

    (the cell and the halves of W are those of the TreeRNN; the paper gives no equations for such a model, these
    are the smallest ones that make the Switch of `expand` read a vector value).  Returns the state of the
    generated tree's root.  `log`, if a dict, receives "expand" / "child" invocation counts and "margin": the
    smallest |W_s[0].h + b_s[0]| over the invocations whose gate decided (d < D) -- how far the nearest decision
    was from flipping."""
    P = _f64(params)
    H = P["W"].shape[0]
    WL, WR = P["W"][:, :H], P["W"][:, H:]
    if log is not None:
        log.setdefault("expand", 0)
        log.setdefault("child", 0)
        log.setdefault("margin", np.inf)

    def expand(h, d):
        g = float(P["W_s"][0] @ h + P["b_s"][0])
        if log is not None:
            log["expand"] += 1
            if d < depth_limit:
                log["margin"] = min(log["margin"], abs(g))
        if d >= depth_limit or g > 0:
            return h
        if log is not None:
            log["child"] += 2
        hl = np.tanh(WL @ h + P["b"])
        hr = np.tanh(WR @ h + P["b"])
        return rnn_cell(P, expand(hl, d + 1), expand(hr, d + 1))

    return deep(expand, P["E"][tok], 0)


def node_loss(h, P, label):
    """-log softmax(W_s h + b_s)[label]"""
    z = P["W_s"] @ h + P["b_s"]
    e = np.exp(z)
    return -np.log(e[label] / e.sum())


def forward(tb, params, cell="rnn", trees=None, with_loss=False, keep=False):
    """Root states of the trees `trees` (default all), [len(trees), H]; with
    `with_loss` also the loss summed over every node of those trees; with
    `keep` also {node: state} for every node visited."""
    P = _f64(params)
    trees = range(tb.B) if trees is None else trees

    def work():
        roots, loss, store = [], 0.0, {}
        for t in trees:
            r = int(tb.tree_root[t])
            if cell == "rnn":
                roots.append(treernn_h(tb, P, r, store))
            else:
                roots.append(treelstm_hc(tb, P, r, store)[0])
        if with_loss:
            for v, s in store.items():
                h = s if cell == "rnn" else s[0]
                loss += node_loss(h, P, int(tb.label[v]))
        return np.array(roots), loss, store

    roots, loss, store = deep(work)
    out = [roots]
    if with_loss:
        out.append(loss)
    if keep:
        out.append(store)
    return out[0] if len(out) == 1 else tuple(out)


# --------------------------------------------------------------------------
# tree networks, loss and gradient by reverse recursion
# --------------------------------------------------------------------------
def _head_backward(h, P, label, G):
    """Gradient operator of the loss head: accumulates dW_s, db_s and returns
    the contribution W_s^T (softmax - onehot) to dh."""
    z = P["W_s"] @ h + P["b_s"]
    e = np.exp(z)
    p = e / e.sum()
    p[label] -= 1.0
    G["W_s"] += np.outer(p, h)
    G["b_s"] += p
    return P["W_s"].T @ p


def _rnn_back(tb, P, G, S, v, dh_in):
    h = S[v]
    dh = dh_in + _head_backward(h, P, int(tb.label[v]), G)
    if tb.left[v] < 0:
        G["E"][tb.tok[v]] += dh
        return
    l, r = int(tb.left[v]), int(tb.right[v])
    x = np.concatenate([S[l], S[r]])
    dz = dh * (1.0 - h * h)
    G["W"] += np.outer(dz, x)
    G["b"] += dz
    dx = P["W"].T @ dz
    H = h.shape[0]
    _rnn_back(tb, P, G, S, l, dx[:H])
    _rnn_back(tb, P, G, S, r, dx[H:])


def _lstm_back(tb, P, G, S, v, dh_in, dc_in):
    h, c = S[v]
    H = h.shape[0]
    dh = dh_in + _head_backward(h, P, int(tb.label[v]), G)
    tc = np.tanh(c)
    if tb.left[v] < 0:
        e = P["E"][tb.tok[v]]
        g = P["W_x"] @ e + P["b_x"]
        i, o, u = sigmoid(g[:H]), sigmoid(g[H:2 * H]), np.tanh(g[2 * H:])
        dc = dc_in + dh * o * (1.0 - tc * tc)
        dg = np.concatenate([dc * u * i * (1 - i), dh * tc * o * (1 - o), dc * i * (1 - u * u)])
        G["W_x"] += np.outer(dg, e)
        G["b_x"] += dg
        G["E"][tb.tok[v]] += P["W_x"].T @ dg
        return
    l, r = int(tb.left[v]), int(tb.right[v])
    (hl, cl), (hr, cr) = S[l], S[r]
    x = np.concatenate([hl, hr])
    g = P["W"] @ x + P["b"]
    i, fl, fr, o = (sigmoid(g[k * H:(k + 1) * H]) for k in range(4))
    u = np.tanh(g[4 * H:])
    dc = dc_in + dh * o * (1.0 - tc * tc)
    dg = np.concatenate([dc * u * i * (1 - i), dc * cl * fl * (1 - fl), dc * cr * fr * (1 - fr),
                         dh * tc * o * (1 - o), dc * i * (1 - u * u)])
    G["W"] += np.outer(dg, x)
    G["b"] += dg
    dx = P["W"].T @ dg
    _lstm_back(tb, P, G, S, l, dx[:H], dc * fl)
    _lstm_back(tb, P, G, S, r, dx[H:], dc * fr)


def loss_and_grad(tb, params, cell="rnn", trees=None):
    """L = sum over the trees `trees` and over every node v of
    -log softmax(W_s h(v) + b_s)[label v]; returns (L, {param: dL/dparam},
    root states).  fp64."""
    P = _f64(params)
    trees = range(tb.B) if trees is None else trees

    def work():
        G = {k: np.zeros_like(v) for k, v in P.items()}
        loss, roots = 0.0, []
        H = P["W_s"].shape[1]
        for t in trees:
            S = {}
            r = int(tb.tree_root[t])
            if cell == "rnn":
                roots.append(treernn_h(tb, P, r, S))
                loss += sum(node_loss(h, P, int(tb.label[v])) for v, h in S.items())
                _rnn_back(tb, P, G, S, r, np.zeros(H))
            else:
                roots.append(treelstm_hc(tb, P, r, S)[0])
                loss += sum(node_loss(s[0], P, int(tb.label[v])) for v, s in S.items())
                _lstm_back(tb, P, G, S, r, np.zeros(H), np.zeros(H))
        return loss, G, np.array(roots)

    return deep(work)


# --------------------------------------------------------------------------
# the same over a pool of processes (trees are independent; sums add up)
# --------------------------------------------------------------------------
def _pool_job(args):
    tb, params, cell, trees = args
    try:                                  # one BLAS thread per worker: the pool already uses every core
        from threadpoolctl import threadpool_limits
        with threadpool_limits(limits=1):
            return loss_and_grad(tb, params, cell, trees)
    except ImportError:
        return loss_and_grad(tb, params, cell, trees)


def loss_and_grad_pool(tb, params, cell="rnn", workers=8, trees=None):
    """loss_and_grad over `workers` spawned processes, each taking a
    contiguous share of the trees; partial losses and gradients are added in
    share order.  Spawn (not fork) so that it is safe after CUDA start-up."""
    import multiprocessing as mp

    trees = list(range(tb.B) if trees is None else trees)
    workers = max(1, min(workers, len(trees)))
    # balance by node count
    sizes = tb.tree_sizes()[trees]
    bounds = np.searchsorted(np.cumsum(sizes), np.linspace(0, sizes.sum(), workers + 1)[1:-1])
    shares = [s.tolist() for s in np.split(np.array(trees), bounds) if len(s)]
    with mp.get_context("spawn").Pool(len(shares)) as pool:
        parts = pool.map(_pool_job, [(tb, params, cell, s) for s in shares])
    loss = sum(p[0] for p in parts)
    G = {k: sum(p[1][k] for p in parts) for k in parts[0][1]}
    roots = np.concatenate([p[2] for p in parts])
    return loss, G, roots
