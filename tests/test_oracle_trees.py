"""Pins for the floating-point side of the CPU oracle (tree networks, loss and
gradients) against library routines, closed-form special cases, brute force on
tiny trees, finite differences and an autograd engine."""
import numpy as np
import pytest
import scipy.special
import torch

import workloads
from oracle import direct, programs, tagged, transform


def _tiny(seed=3, H=6, V=11, cell="rnn", B=5, max_leaves=5):
    rng = np.random.default_rng(seed)
    shapes = [workloads.random_split_shape(rng, int(L)) for L in rng.integers(1, max_leaves + 1, size=B)]
    tb = workloads.tree_batch_from_shapes(shapes, seed, vocab=V)
    mk = workloads.treernn_params if cell == "rnn" else workloads.treelstm_params
    p = mk(seed, V, H, H)
    # non-zero biases so that a dropped bias term shows
    for k in p:
        if k.startswith("b"):
            p[k] = (0.3 * rng.standard_normal(p[k].shape)).astype(np.float32)
    return tb, p


def _P(p):
    return {k: np.asarray(v, dtype=np.float64) for k, v in p.items()}


# --------------------------------------------------------------------------
# cells against library routines
# --------------------------------------------------------------------------
def test_rnn_cell_is_torch_rnncell():
    """tanh(W [h_l; h_r] + b) is an Elman cell with hidden = h_l, input = h_r."""
    _, p = _tiny(H=7)
    P = _P(p)
    H = 7
    rng = np.random.default_rng(0)
    hl, hr = rng.standard_normal(H), rng.standard_normal(H)
    m = torch.nn.RNNCell(H, H, nonlinearity="tanh").double()
    with torch.no_grad():
        m.weight_hh.copy_(torch.tensor(P["W"][:, :H]))
        m.weight_ih.copy_(torch.tensor(P["W"][:, H:]))
        m.bias_hh.copy_(torch.tensor(P["b"]))
        m.bias_ih.zero_()
        want = m(torch.tensor(hr)[None], torch.tensor(hl)[None])[0].numpy()
    np.testing.assert_allclose(direct.rnn_cell(P, hl, hr), want, rtol=0, atol=1e-14)
    ops = programs.tree_net_ops(None, p, "rnn")
    np.testing.assert_allclose(ops["cell_rnn"](hl, hr), want, rtol=0, atol=1e-14)


def _torch_lstm(H, Wi, Wh, b, order):
    """torch.nn.LSTMCell with its gate rows (i, f, g, o) filled from blocks
    named in `order` (a dict gate -> (rows of Wi, rows of Wh, rows of b) or None for zeros)."""
    m = torch.nn.LSTMCell(Wi.shape[1], H).double()
    with torch.no_grad():
        m.bias_hh.zero_()
        for k, gate in enumerate("ifgo"):
            sl = slice(k * H, (k + 1) * H)
            src = order[gate]
            if src is None:
                m.weight_ih[sl].zero_(); m.weight_hh[sl].zero_(); m.bias_ih[sl].zero_()
            else:
                m.weight_ih[sl].copy_(torch.tensor(Wi[src])); m.weight_hh[sl].copy_(torch.tensor(Wh[src]))
                m.bias_ih[sl].copy_(torch.tensor(b[src]))
    return m


def test_lstm_cell_reduces_to_torch_lstmcell():
    """With c_r = 0 the binary cell is a standard LSTM cell with hidden state
    (h_l, c_l), input h_r and gates (i, f, g, o) = (i, f_l, u, o); mirrored
    with c_l = 0.  Together the two cases pin every row block of W."""
    _, p = _tiny(H=5, cell="lstm")
    P = _P(p)
    H = 5
    rng = np.random.default_rng(1)
    hl, cl, hr, cr = (rng.standard_normal(H) for _ in range(4))
    blk = lambda k: slice(k * H, (k + 1) * H)  # noqa: E731
    Wl, Wr = P["W"][:, :H], P["W"][:, H:]
    # c_r = 0: hidden = left, input = right
    m = _torch_lstm(H, Wr, Wl, P["b"], {"i": blk(0), "f": blk(1), "g": blk(4), "o": blk(3)})
    with torch.no_grad():
        h_t, c_t = m(torch.tensor(hr)[None], (torch.tensor(hl)[None], torch.tensor(cl)[None]))
    h, c = direct.lstm_cell(P, hl, cl, hr, np.zeros(H))
    np.testing.assert_allclose(h, h_t[0].numpy(), atol=1e-14)
    np.testing.assert_allclose(c, c_t[0].numpy(), atol=1e-14)
    # c_l = 0: hidden = right, input = left, forget gate = f_r
    m = _torch_lstm(H, Wl, Wr, P["b"], {"i": blk(0), "f": blk(2), "g": blk(4), "o": blk(3)})
    with torch.no_grad():
        h_t, c_t = m(torch.tensor(hl)[None], (torch.tensor(hr)[None], torch.tensor(cr)[None]))
    h, c = direct.lstm_cell(P, hl, np.zeros(H), hr, cr)
    np.testing.assert_allclose(h, h_t[0].numpy(), atol=1e-14)
    np.testing.assert_allclose(c, c_t[0].numpy(), atol=1e-14)
    # additivity in the two forget paths gives the general case
    h_full, c_full = direct.lstm_cell(P, hl, cl, hr, cr)
    c_a = direct.lstm_cell(P, hl, cl, hr, np.zeros(H))[1]
    c_b = direct.lstm_cell(P, hl, np.zeros(H), hr, cr)[1]
    c_0 = direct.lstm_cell(P, hl, np.zeros(H), hr, np.zeros(H))[1]
    np.testing.assert_allclose(c_full, c_a + c_b - c_0, atol=1e-14)
    # the interpreter's operator table is typed separately: same values
    ops = programs.tree_net_ops(None, p, "lstm")
    h2, c2 = ops["cell_lstm"]((hl, cl), (hr, cr))
    np.testing.assert_allclose(h2, h_full, atol=1e-14)
    np.testing.assert_allclose(c2, c_full, atol=1e-14)


def test_lstm_leaf_is_lstmcell_from_zero_state():
    _, p = _tiny(H=5, cell="lstm")
    P = _P(p)
    H = 5
    blk = lambda k: slice(k * H, (k + 1) * H)  # noqa: E731
    e = np.random.default_rng(2).standard_normal(H)
    m = _torch_lstm(H, P["W_x"], np.zeros((3 * H, H)), P["b_x"], {"i": blk(0), "f": None, "g": blk(2), "o": blk(1)})
    with torch.no_grad():
        h_t, c_t = m(torch.tensor(e)[None], (torch.zeros(1, H).double(), torch.zeros(1, H).double()))
    h, c = direct.lstm_leaf(P, e)
    np.testing.assert_allclose(h, h_t[0].numpy(), atol=1e-14)
    np.testing.assert_allclose(c, c_t[0].numpy(), atol=1e-14)


def test_loss_head_against_logsumexp():
    _, p = _tiny()
    P = _P(p)
    h = np.random.default_rng(4).standard_normal(6)
    z = P["W_s"] @ h + P["b_s"]
    for lab in range(5):
        want = scipy.special.logsumexp(z) - z[lab]
        assert abs(direct.node_loss(h, P, lab) - want) < 1e-13
        assert abs(programs.node_loss_value(h, P["W_s"], P["b_s"], lab) - want) < 1e-13
    # uniform logits: loss = log 5
    P0 = dict(P, W_s=np.zeros_like(P["W_s"]), b_s=np.zeros(5))
    assert abs(direct.node_loss(h, P0, 3) - np.log(5)) < 1e-14


# --------------------------------------------------------------------------
# whole trees: brute force, special cases, tagged == direct
# --------------------------------------------------------------------------
def test_treernn_brute_force_nested_expression():
    """A 4-leaf tree ((a b) (c d)) and a 3-leaf chain ((a b) c), written out."""
    _, p = _tiny(H=6, V=11)
    P = _P(p)
    E, W, b = P["E"], P["W"], P["b"]
    cell = lambda x, y: np.tanh(W @ np.concatenate([x, y]) + b)  # noqa: E731
    # tree 0: nodes 0=(1,4) 1=(2,3) 2=leaf 3=leaf 4=(5,6) 5=leaf 6=leaf ; tree 1: 7=(8,11) 8=(9,10) 9,10,11 leaves
    left = np.array([1, 2, -1, -1, 5, -1, -1, 8, 9, -1, -1, -1], dtype=np.int32)
    right = np.array([4, 3, -1, -1, 6, -1, -1, 11, 10, -1, -1, -1], dtype=np.int32)
    tok = np.array([-1, -1, 3, 7, -1, 0, 10, -1, -1, 5, 5, 2], dtype=np.int32)
    tb = workloads.TreeBatch(np.array([0, 7], dtype=np.int32), left, right, tok, np.zeros(12, dtype=np.int32))
    want0 = cell(cell(E[3], E[7]), cell(E[0], E[10]))
    want1 = cell(cell(E[5], E[5]), E[2])
    got = direct.forward(tb, p, "rnn")
    np.testing.assert_allclose(got[0], want0, atol=1e-15)
    np.testing.assert_allclose(got[1], want1, atol=1e-15)
    # swapping the children changes the result (operand order is pinned)
    assert np.abs(cell(E[2], cell(E[5], E[5])) - want1).max() > 1e-3


def test_treernn_special_cases():
    tb, p = _tiny(B=8, max_leaves=6)
    P = _P(p)
    # single-leaf tree: the root state is the embedding row, exactly
    one = workloads.tree_batch_from_shapes([workloads.random_split_shape(np.random.default_rng(0), 1)], 5, vocab=11)
    assert np.array_equal(direct.forward(one, p, "rnn")[0], P["E"][one.tok[0]])
    # W = 0: every internal state is tanh(b)
    p0 = dict(p, W=np.zeros_like(p["W"]))
    _, _, store = direct.forward(tb, p0, "rnn", with_loss=True, keep=True)
    for v, h in store.items():
        if tb.left[v] >= 0:
            np.testing.assert_allclose(h, np.tanh(P["b"]), atol=1e-15)
    # equal leaves on a perfect tree: one vector recurrence per level
    pt = workloads.tree_batch_from_shapes([workloads.perfect_tree_shape(4)], 5, vocab=11)
    pt.tok[pt.left < 0] = 4
    h = P["E"][4]
    for _ in range(4):
        h = np.tanh(P["W"] @ np.concatenate([h, h]) + P["b"])
    np.testing.assert_allclose(direct.forward(pt, p, "rnn")[0], h, atol=1e-15)


def test_lstm_zero_weights_closed_form():
    """W = 0, b = 0: all gates 1/2 and u = 0, so c = (c_l + c_r)/2, h = tanh(c)/2."""
    tb, p = _tiny(cell="lstm", B=6, max_leaves=6)
    p0 = dict(p, W=np.zeros_like(p["W"]), b=np.zeros_like(p["b"]))
    _, _, store = direct.forward(tb, p0, "lstm", with_loss=True, keep=True)
    for v, (h, c) in store.items():
        if tb.left[v] >= 0:
            cl, cr = store[int(tb.left[v])][1], store[int(tb.right[v])][1]
            np.testing.assert_allclose(c, 0.5 * (cl + cr), atol=1e-15)
            np.testing.assert_allclose(h, 0.5 * np.tanh(c), atol=1e-15)


@pytest.mark.parametrize("cell", ["rnn", "lstm"])
def test_tagged_interpreter_equals_direct_recursion(cell):
    tb, p = _tiny(cell=cell, B=6, max_leaves=7, seed=9)
    ops = programs.tree_net_ops(tb, p, cell)
    g = transform.transform(programs.tree_net_program(cell, with_loss=False))
    gl = transform.transform(programs.tree_net_program(cell, with_loss=True))
    roots, loss, store = direct.forward(tb, p, cell, with_loss=True, keep=True)
    total = 0.0
    for t in range(tb.B):
        root = int(tb.tree_root[t])
        r = tagged.run(g, {0: root}, ops)
        val = r.value if cell == "rnn" else r.value[0]
        np.testing.assert_allclose(val, roots[t], rtol=0, atol=1e-12)
        assert r.leftover == 0
        # every invocation's returned state equals direct recursion at its node
        for tag, arg in r.calls.items():
            got = r.returns[tag] if cell == "rnn" else r.returns[tag][0]
            want = store[arg[0]] if cell == "rnn" else store[arg[0]][0]
            np.testing.assert_allclose(got, want, rtol=0, atol=1e-12)
        rl = tagged.run(gl, {0: root}, ops, dead_tokens=False)
        state, l = rl.value
        total += l
        np.testing.assert_allclose(state if cell == "rnn" else state[0], roots[t], rtol=0, atol=1e-12)
    assert abs(total - loss) < 1e-10 * max(1.0, abs(loss))


# --------------------------------------------------------------------------
# gradients
# --------------------------------------------------------------------------
def _total_loss(tb, p, cell):
    return direct.forward(tb, p, cell, with_loss=True)[1]


@pytest.mark.parametrize("cell", ["rnn", "lstm"])
def test_gradient_by_central_differences(cell):
    tb, p = _tiny(cell=cell, B=4, max_leaves=5, seed=11)
    p = {k: v.astype(np.float64) for k, v in p.items()}
    loss, G, _ = direct.loss_and_grad(tb, p, cell)
    assert abs(loss - _total_loss(tb, p, cell)) < 1e-12 * abs(loss)
    rng = np.random.default_rng(0)
    eps = 1e-5
    used = np.unique(tb.tok[tb.tok >= 0])
    for name, g in G.items():
        picks = []
        if name == "E":
            picks = [(int(r), int(c)) for r in used[:3] for c in rng.integers(0, g.shape[1], 3)]
            unused = [r for r in range(g.shape[0]) if r not in set(used.tolist())]
            if unused:
                assert np.all(g[unused] == 0)
        else:
            flat = rng.choice(g.size, size=min(g.size, 25), replace=False)
            picks = [np.unravel_index(i, g.shape) for i in flat]
        for idx in picks:
            q = {k: v.copy() for k, v in p.items()}
            q[name][idx] += eps
            up = _total_loss(tb, q, cell)
            q[name][idx] -= 2 * eps
            dn = _total_loss(tb, q, cell)
            fd = (up - dn) / (2 * eps)
            assert abs(fd - g[idx]) <= 1e-6 * max(1.0, abs(fd)), (name, idx, fd, g[idx])


def _torch_tree_loss(tb, T, cell):
    """The same loss assembled from torch operations, for its autograd."""
    H = T["W_s"].shape[1]
    total = 0.0

    def state(v):
        nonlocal total
        if tb.left[v] < 0:
            e = T["E"][int(tb.tok[v])]
            if cell == "rnn":
                s = (e, None)
            else:
                g = T["W_x"] @ e + T["b_x"]
                c = torch.sigmoid(g[:H]) * torch.tanh(g[2 * H:])
                s = (torch.sigmoid(g[H:2 * H]) * torch.tanh(c), c)
        else:
            (hl, cl), (hr, cr) = state(int(tb.left[v])), state(int(tb.right[v]))
            g = T["W"] @ torch.cat([hl, hr]) + T["b"]
            if cell == "rnn":
                s = (torch.tanh(g), None)
            else:
                i, fl, fr, o, u = g.split(H)
                c = torch.sigmoid(i) * torch.tanh(u) + torch.sigmoid(fl) * cl + torch.sigmoid(fr) * cr
                s = (torch.sigmoid(o) * torch.tanh(c), c)
        total = total + torch.nn.functional.cross_entropy((T["W_s"] @ s[0] + T["b_s"])[None],
                                                          torch.tensor([int(tb.label[v])]), reduction="sum")
        return s

    roots = [state(int(r))[0] for r in tb.tree_root]
    return total, roots


@pytest.mark.parametrize("cell", ["rnn", "lstm"])
def test_gradient_against_autograd(cell):
    tb, p = _tiny(cell=cell, B=6, max_leaves=8, seed=21, H=8, V=13)
    T = {k: torch.tensor(v, dtype=torch.float64, requires_grad=True) for k, v in p.items()}
    total, roots = _torch_tree_loss(tb, T, cell)
    total.backward()
    loss, G, r = direct.loss_and_grad(tb, p, cell)
    assert abs(loss - total.item()) < 1e-11 * abs(loss)
    np.testing.assert_allclose(r, torch.stack(roots).detach().numpy(), atol=1e-13)
    for k in G:
        np.testing.assert_allclose(G[k], T[k].grad.numpy(), rtol=0, atol=1e-11 * max(1.0, np.abs(G[k]).max()))


def test_head_gradient_sums_to_zero_and_pool_matches_serial():
    tb, p = _tiny(B=7, max_leaves=6, seed=5)
    loss, G, roots = direct.loss_and_grad(tb, p, "rnn")
    # softmax - onehot sums to zero per node, hence db_s sums to zero
    assert abs(G["b_s"].sum()) < 1e-12
    loss2, G2, roots2 = direct.loss_and_grad_pool(tb, p, "rnn", workers=3)
    assert abs(loss - loss2) < 1e-12 * abs(loss)
    np.testing.assert_allclose(roots, roots2, atol=0)
    for k in G:
        np.testing.assert_allclose(G[k], G2[k], rtol=0, atol=1e-13)


def test_deep_chain_recursion_runs():
    tb = workloads.tree_batch_from_shapes([workloads.chain_tree_shape(3000)], 2, vocab=50)
    p = workloads.treernn_params(2, 50, 8, 8)
    loss, G, roots = direct.loss_and_grad(tb, p, "rnn")
    assert np.isfinite(loss) and np.all(np.isfinite(G["W"])) and roots.shape == (1, 8)
