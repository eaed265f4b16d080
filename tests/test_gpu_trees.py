"""GPU parity, recursive tree networks: root states, loss and parameter
gradients of the CUDA executor against the fp64 CPU oracle, through the C
boundary.  Tolerance (tensor-normalised max error, per output tensor):
1e-4 for fp32 arithmetic, 2e-2 for bf16 operands with fp32 accumulation."""
import os

import numpy as np
import pytest

import workloads
import paper_2410_20225_b200 as rdf
from oracle import direct

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

TOL = {rdf.F32: 1e-4, rdf.BF16: 2e-2}
WORKERS = max(1, min(32, (os.cpu_count() or 2) - 1))


def relerr(got, want):
    want = np.asarray(want, dtype=np.float64)
    got = np.asarray(got, dtype=np.float64)
    return float(np.abs(got - want).max() / max(np.abs(want).max(), 1e-30))


def graph(cell="rnn", with_loss=False):
    fs, r = rdf.tree_net_program(cell, with_loss)
    return rdf.Graph(fs, r, rdf.TAGS_FRAME)


def check_forward(cfg, compute=rdf.F32, trees=None, cell="rnn"):
    tb, p = cfg["trees"], cfg["params"]
    g = graph(cell)
    h, _ = g.eval_trees(rdf.Graph.device_trees(tb), rdf.Graph.device_params(p), compute)
    h = h.cpu().numpy()
    st = g.stats()
    assert st["invocations"] == tb.N and st["cells"] == tb.n_cells and st["leaves"] == tb.N - tb.n_cells
    trees = list(range(tb.B)) if trees is None else trees
    want = direct.forward(tb, p, cell, trees=trees)
    assert relerr(h[trees], want) <= TOL[compute]
    return st


def check_embedding_rows(tb, dE, want, tol):
    """The embedding gradient row by row (one maximum over the whole table would hide a wrong row): the rows of
    tokens that no leaf carries are exactly zero, and every other row is within the tolerance of the larger of
    its own largest entry and a floor of 5 % of the table's largest entry (a row whose contributions cancel
    is small against the values that were rounded on the way to it)."""
    dE = np.asarray(dE, dtype=np.float64)
    touched = np.zeros(dE.shape[0], dtype=bool)
    touched[tb.tok[tb.left < 0]] = True
    assert not dE[~touched].any()
    scale = np.maximum(np.abs(want[touched]).max(axis=1), 0.05 * np.abs(want).max())
    row_err = np.abs(dE[touched] - want[touched]).max(axis=1) / scale
    assert row_err.max() <= tol, float(row_err.max())
    return float(row_err.max())


_ORACLE_CACHE = {}


def oracle_grad(name, cfg, cell, workers):
    """loss, gradients and root states of the fp64 oracle for a named full-size workload (computed once)."""
    if name not in _ORACLE_CACHE:
        tb, p = cfg["trees"], cfg["params"]
        _ORACLE_CACHE[name] = (direct.loss_and_grad_pool(tb, p, cell, workers=workers) if workers > 1
                               else direct.loss_and_grad(tb, p, cell))
    return _ORACLE_CACHE[name]


def check_grad(cfg, compute=rdf.F32, workers=1, cell="rnn", name=None):
    tb, p = cfg["trees"], cfg["params"]
    g = graph(cell, with_loss=True)
    loss, h, grads = g.grad_trees(rdf.Graph.device_trees(tb), rdf.Graph.device_params(p), compute)
    st = g.stats()
    assert st["status"] == 0 and st["invocations"] == tb.N
    if name is not None:
        want_loss, G, roots = oracle_grad(name, cfg, cell, workers)
    elif workers > 1:
        want_loss, G, roots = direct.loss_and_grad_pool(tb, p, cell, workers=workers)
    else:
        want_loss, G, roots = direct.loss_and_grad(tb, p, cell)
    tol = TOL[compute]
    assert relerr(h.cpu().numpy(), roots) <= tol
    assert abs(loss.item() - want_loss) <= tol * abs(want_loss)
    errs = {k: relerr(grads[k].cpu().numpy(), G[k]) for k in G}
    assert all(e <= tol for e in errs.values()), errs
    errs["E rows"] = check_embedding_rows(tb, grads["E"].cpu().numpy(), G["E"], tol)
    return st, errs


def test_treernn_forward_config2_full():
    st = check_forward(workloads.config(2))
    assert st["waves"] <= 2 * 32 + 8


def test_single_leaf_trees_and_tiny_batches():
    rng = np.random.default_rng(0)
    for Ls in ([1], [1, 1, 1], [2], [1, 3, 1, 2]):
        tb = workloads.tree_batch_from_shapes([workloads.random_split_shape(rng, L) for L in Ls], 7, vocab=50)
        p = workloads.treernn_params(7, 50, 8, 8)
        p["b"] = (0.2 * rng.standard_normal(8)).astype(np.float32)
        cfg = {"trees": tb, "params": p}
        check_forward(cfg)
        check_grad(cfg)
    # a single leaf: the root state is the embedding row, exactly
    tb = workloads.tree_batch_from_shapes([workloads.random_split_shape(rng, 1)], 7, vocab=50)
    h, _ = graph().eval_trees(rdf.Graph.device_trees(tb), rdf.Graph.device_params(p))
    assert np.array_equal(h.cpu().numpy()[0], p["E"][tb.tok[0]])


def test_tags_of_tree_invocations():
    """Frame ids decode (through the parent links) to the label lists of direct recursion."""
    tb = workloads.config(2, B=40)["trees"]
    p = workloads.treernn_params(1, 1000, 64, 64)
    g = graph()
    _, tr = g.eval_trees(rdf.Graph.device_trees(tb), rdf.Graph.device_params(p), trace_capacity=2 * tb.N)
    calls = tr[tr["kind"] == 0]
    assert len(calls) == tb.N
    parent = dict(zip(calls["tag"].tolist(), calls["parent"].tolist()))
    label = dict(zip(calls["tag"].tolist(), calls["label"].tolist()))
    node = dict(zip(calls["tag"].tolist(), calls["value"].tolist()))
    got = set()
    for f in parent:
        labs, q = [], f
        while q >= tb.B:
            labs.append(label[q])
            q = parent[q]
        got.add((q, tuple(labs), node[f]))
    want = set()
    for t in range(tb.B):
        for tag, v in direct.deep(direct.tree_invocations, tb, int(tb.tree_root[t])):
            want.add((t, tag, v))
    assert got == want


def test_frame_ids_are_handed_out_in_wave_order():
    """The gradient pass walks frame-id ranges: every frame must have a larger id than any frame of a
    shallower call depth (ids are interned wave by wave, a call fires one wave after its caller)."""
    tb = workloads.config(3, B=64, V=300, H=32)["trees"]
    p = workloads.treernn_params(2, 300, 32, 32)
    g = graph()
    _, tr = g.eval_trees(rdf.Graph.device_trees(tb), rdf.Graph.device_params(p), trace_capacity=2 * tb.N)
    calls = tr[tr["kind"] == 0]
    frames = calls["tag"].astype(np.int64)
    parents = calls["parent"].astype(np.int64)
    assert sorted(frames.tolist()) == list(range(tb.B, tb.B + tb.N))        # ids B .. B + N - 1, each once
    depth = np.zeros(tb.B + tb.N, dtype=np.int64)
    for f, q in sorted(zip(frames.tolist(), parents.tolist())):             # a parent's id is smaller: already done
        assert q < f
        depth[f] = depth[q] + 1
    d = depth[tb.B:]
    assert np.all(np.diff(d) >= 0)                                          # depth never decreases with the id


def test_treernn_grad_small_fp32():
    cfg = workloads.config(3, B=96, V=500, H=64)
    cfg["params"] = workloads.treernn_params(5, 500, 64, 64)
    rng = np.random.default_rng(1)
    cfg["params"]["b"] = (0.1 * rng.standard_normal(64)).astype(np.float32)
    cfg["params"]["b_s"] = (0.1 * rng.standard_normal(5)).astype(np.float32)
    check_grad(cfg)


def test_treernn_grad_ragged_hidden_size():
    """H = 300 is not a multiple of the tile sizes: ragged tiles in every contraction."""
    cfg = workloads.config(3, B=64, V=700, H=300)
    cfg["params"] = workloads.treernn_params(5, 700, 300, 300)
    check_grad(cfg)


@pytest.mark.parametrize("H", [64, 300])
def test_treernn_bf16_tensor_core_path(H):
    """bf16 operands on the tensor cores (fp32 accumulation): parameters are bf16-representable,
    states are rounded to bf16 after every cell; tolerance 2e-2."""
    cfg = workloads.config(3, B=200, V=900, H=H)
    check_forward(cfg, rdf.BF16)
    check_grad(cfg, rdf.BF16)
    # more than one 128-row tile per wave and a ragged last tile
    cfg = workloads.config(3, B=700, V=900, H=H)
    st = check_forward(cfg, rdf.BF16)
    assert st["cells"] > 3 * 128


@pytest.mark.parametrize("H", [100, 256])
def test_treernn_bf16_padding_and_biases(H):
    """H = 100 leaves 28 pad columns in the bf16 state rows (the first of them holds the constant input from
    which the bias gradient is contracted); H = 256 leaves none (the bias gradient is a column sum then).
    Nonzero biases; several tiles per wave."""
    cfg = workloads.config(3, B=300, V=500, H=H)
    rng = np.random.default_rng(11)
    cfg["params"]["b"] = workloads.bf16_round((0.2 * rng.standard_normal(H)).astype(np.float32))
    cfg["params"]["b_s"] = workloads.bf16_round((0.2 * rng.standard_normal(5)).astype(np.float32))
    check_forward(cfg, rdf.BF16)
    check_grad(cfg, rdf.BF16)


def test_treernn_bf16_tiny_and_all_leaf_batches():
    """The tensor-core path on degenerate batches: a single leaf, only leaves (no cell at all: every contraction of
    the gradient pass is empty), one cell, a handful of small trees."""
    rng = np.random.default_rng(3)
    p = workloads.treernn_params(9, 60, 64, 64, bf16=True)
    p["b"] = workloads.bf16_round((0.2 * rng.standard_normal(64)).astype(np.float32))
    for Ls in ([1], [1, 1, 1, 1], [2], [1, 3, 1, 2, 5]):
        tb = workloads.tree_batch_from_shapes([workloads.random_split_shape(rng, L) for L in Ls], 7, vocab=60)
        cfg = {"trees": tb, "params": p}
        check_forward(cfg, rdf.BF16)
        check_grad(cfg, rdf.BF16)


def test_depth_stress_reduced():
    cfg = workloads.config(5, chains=3, chain_depth=300, perfect=2, perfect_height=7, V=400, H=32)
    st, _ = check_grad(cfg)
    assert st["waves"] >= 2 * 300 and st["waves_backward"] >= 300


def test_frame_tags_required_for_depth():
    """The packed path form cannot hold a depth-300 tag: the integer fold over a chain
    reports overflow in path form and runs in frame form."""
    tb = workloads.tree_batch_from_shapes([workloads.chain_tree_shape(300)], 3, vocab=10)
    dt = rdf.Graph.device_trees(tb)
    fs, r = rdf.tree_fold_program("height")
    with pytest.raises(rdf.RdfError) as e:
        rdf.Graph(fs, r, rdf.TAGS_PATH).eval_trees(dt, None)
    assert e.value.code == -4
    y, _ = rdf.Graph(fs, r, rdf.TAGS_FRAME).eval_trees(dt, None)
    assert y.item() == 300


@pytest.mark.parametrize("compute", [rdf.F32, rdf.BF16])
def test_undersized_capacity_is_a_status_code_for_tree_networks(compute):
    """A frame table too small for the batch: the scheduler reports RDF_ERR_FRAMES_FULL, every later kernel
    of the call does nothing, and the same graph runs a correctly sized call afterwards."""
    cfg = workloads.config(3, B=40, V=300, H=64)
    tb, p = cfg["trees"], cfg["params"]
    dt, dp = rdf.Graph.device_trees(tb), rdf.Graph.device_params(p)
    g = graph("rnn", with_loss=True)
    with pytest.raises(rdf.RdfError) as e:
        g.grad_trees(dt, dp, compute, max_invocations=tb.N // 3)
    assert e.value.code == -6                     # RDF_ERR_FRAMES_FULL
    ge = graph("rnn")
    with pytest.raises(rdf.RdfError) as e:
        ge.eval_trees(dt, dp, compute, max_invocations=tb.N // 3)
    assert e.value.code == -6
    loss, h, grads = g.grad_trees(dt, dp, compute)
    want_loss, G, roots = direct.loss_and_grad(tb, p, "rnn")
    assert relerr(h.cpu().numpy(), roots) <= TOL[compute]
    assert abs(loss.item() - want_loss) <= TOL[compute] * abs(want_loss)
    assert all(relerr(grads[k].cpu().numpy(), G[k]) <= TOL[compute] for k in G)


def test_treernn_config3_full_size():
    """8192 trees, H = 300, fwd + bwd at full size; the oracle runs over a pool of processes."""
    cfg = workloads.config(3)
    compute = rdf.BF16
    st, errs = check_grad(cfg, compute, workers=WORKERS, name="config3")
    print("config 3 errors:", errs, st)


@pytest.mark.parametrize("k,cell", [(3, "rnn"), (4, "lstm")])
def test_forward_only_full_size_bf16(k, cell):
    """rdf_eval (forward only: no retained gates, no gradient buffers) on the 8192-tree workloads with bf16
    operands: the root state of every tree against the fp64 oracle."""
    cfg = workloads.config(k)
    tb, p = cfg["trees"], cfg["params"]
    g = graph(cell)
    h, _ = g.eval_trees(rdf.Graph.device_trees(tb), rdf.Graph.device_params(p), rdf.BF16)
    st = g.stats()
    assert st["invocations"] == tb.N and st["cells"] == tb.n_cells and st["leaves"] == tb.N - tb.n_cells
    _, _, roots = oracle_grad("config%d" % k, cfg, cell, WORKERS)
    assert roots.shape == (tb.B, cfg["H"])
    assert relerr(h.cpu().numpy(), roots) <= TOL[rdf.BF16]


def test_bad_indices_in_the_batch_are_a_status_code():
    """A token id outside the embedding table, or a child index outside the node arrays, is reported as
    RDF_ERR_BAD_ARG by the device (the access is skipped, nothing faults), for rdf_eval and rdf_grad, fp32 and
    bf16; the graph runs the intact batch afterwards."""
    cfg = workloads.config(3, B=40, V=300, H=64)
    tb, p = cfg["trees"], cfg["params"]
    dp = rdf.Graph.device_params(p)
    leaf = int(np.flatnonzero(tb.left < 0)[7])
    cell = int(np.flatnonzero(tb.left >= 0)[5])
    g = graph("rnn", with_loss=True)
    ge = graph("rnn")
    for compute in (rdf.F32, rdf.BF16):
        for field, at, value in (("tok", leaf, 300), ("tok", leaf, -5), ("right", cell, tb.N + 3), ("left", cell, 2 ** 30),
                                 ("tree_root", 3, tb.N)):
            dt = rdf.Graph.device_trees(tb)
            dt[field][at] = value
            with pytest.raises(rdf.RdfError) as e:
                g.grad_trees(dt, dp, compute)
            assert e.value.code == -2
            with pytest.raises(rdf.RdfError) as e:
                ge.eval_trees(dt, dp, compute)
            assert e.value.code == -2
        loss, h, grads = g.grad_trees(rdf.Graph.device_trees(tb), dp, compute)
        want_loss, G, roots = direct.loss_and_grad(tb, p, "rnn")
        assert relerr(h.cpu().numpy(), roots) <= TOL[compute]
        assert all(relerr(grads[k].cpu().numpy(), G[k]) <= TOL[compute] for k in G)


def _lstm_cfg(B, V, H, seed=5):
    cfg = workloads.config(4, B=B, V=V, H=H)
    p = workloads.treelstm_params(seed, V, H, H)
    rng = np.random.default_rng(seed)
    for k in ("b", "b_x", "b_s"):
        p[k] = (0.1 * rng.standard_normal(p[k].shape)).astype(np.float32)
    cfg["params"] = p
    return cfg


def test_treelstm_small_and_tiny():
    rng = np.random.default_rng(2)
    for Ls in ([1], [2], [1, 3, 1, 2]):
        tb = workloads.tree_batch_from_shapes([workloads.random_split_shape(rng, L) for L in Ls], 7, vocab=50)
        cfg = {"trees": tb, "params": _lstm_cfg(1, 50, 8)["params"]}
        check_forward(cfg, cell="lstm")
        check_grad(cfg, cell="lstm")
    check_forward(_lstm_cfg(96, 500, 64), cell="lstm")
    check_grad(_lstm_cfg(96, 500, 64), cell="lstm")


def test_treelstm_bf16_tiny_and_all_leaf_batches():
    """The tensor-core TreeLSTM on degenerate batches (a single leaf, only leaves, one cell, a few small trees), with
    H = 64 (no pad column: bias gradients by column sums) and H = 40 (pad columns: bias gradients from the contractions)."""
    rng = np.random.default_rng(4)
    for H in (64, 40):
        p = workloads.treelstm_params(9, 60, H, H, bf16=True)
        for k in ("b", "b_x", "b_s"):
            p[k] = workloads.bf16_round((0.1 * rng.standard_normal(p[k].shape)).astype(np.float32))
        for Ls in ([1], [1, 1, 1, 1], [2], [1, 3, 1, 2, 5]):
            tb = workloads.tree_batch_from_shapes([workloads.random_split_shape(rng, L) for L in Ls], 7, vocab=60)
            cfg = {"trees": tb, "params": p}
            check_forward(cfg, rdf.BF16, cell="lstm")
            check_grad(cfg, rdf.BF16, cell="lstm")


def test_treelstm_ragged_hidden_size():
    check_grad(_lstm_cfg(48, 700, 300), cell="lstm")


@pytest.mark.parametrize("H", [64, 300])
def test_treelstm_bf16_tensor_core_path(H):
    """TreeLSTM with bf16 operands on the tensor cores: weights are bf16-representable, h is rounded to
    bf16 after every cell (c stays fp32); tolerance 2e-2."""
    cfg = workloads.config(4, B=200, V=900, H=H)
    check_forward(cfg, rdf.BF16, cell="lstm")
    check_grad(cfg, rdf.BF16, cell="lstm")
    st = check_forward(workloads.config(4, B=700, V=900, H=H), rdf.BF16, cell="lstm")
    assert st["cells"] > 3 * 128


def test_treelstm_config4_full_size():
    """Binary TreeLSTM, 8192 trees, H = 300, fwd + bwd in the benchmark's launch configuration: loss, the root
    state of every tree and all seven gradients of the full batch against the fp64 oracle (run over a pool of
    processes), element by element.  As an extra, additivity: the gradient of a sum of per-tree losses is the
    sum of the gradients of the two halves of the batch."""
    cfg = workloads.config(4)
    tb, p = cfg["trees"], cfg["params"]
    compute = rdf.BF16
    st, errs = check_grad(cfg, compute, workers=WORKERS, cell="lstm", name="config4")
    print("config 4 errors:", errs)
    assert st["cells"] == tb.n_cells
    g = graph("lstm", with_loss=True)
    dp = rdf.Graph.device_params(p)
    loss, h, grads = g.grad_trees(rdf.Graph.device_trees(tb), dp, compute)
    full = {k: v.cpu().numpy().astype(np.float64) for k, v in grads.items()}
    halves, loss_sum = None, 0.0
    for part in (range(0, tb.B // 2), range(tb.B // 2, tb.B)):
        sub = workloads.subset_trees(tb, list(part))
        l2, _, g2 = g.grad_trees(rdf.Graph.device_trees(sub), dp, compute)
        loss_sum += l2.item()
        cur = {k: v.cpu().numpy().astype(np.float64) for k, v in g2.items()}
        halves = cur if halves is None else {k: halves[k] + cur[k] for k in cur}
    assert abs(loss.item() - loss_sum) <= 1e-4 * abs(loss_sum)
    assert all(relerr(full[k], halves[k]) <= 1e-4 for k in full)


@pytest.mark.parametrize("cell,H", [("rnn", 300), ("rnn", 64), ("lstm", 300), ("lstm", 64)])
def test_bf16_gradient_sums_run_to_run(cell, H):
    """Parameter gradients are sums over every invocation.  By default they are added up with floating-point atomics
    in arrival order: two runs on the same input agree up to the rounding of those sums (bounded here: 1e-5 of the
    largest entry; the tolerance against the oracle is 2e-2), and the root states -- one fixed expression per
    invocation -- agree bit for bit.
    With `reproducible` the cells are put in an order that depends on the input alone (call depth, then node
    index), the floating-point sums run in a fixed order over that order (split-K partial tiles and per-block
    partials added up in sequence) and the sums that many blocks contribute to are exact integer sums in fixed point:
    loss and all gradients are bit-identical from call to call, also from a fresh graph and workspace, and still
    within the tolerance of the oracle.  H = 300 takes the bias gradients out of the weight-gradient contraction,
    H = 64 from column sums."""
    cfg = workloads.config(3 if cell == "rnn" else 4, B=700, V=900, H=H)
    tb, p = cfg["trees"], cfg["params"]
    dt, dp = rdf.Graph.device_trees(tb), rdf.Graph.device_params(p)
    for reproducible in (False, True):
        runs = []
        g = graph(cell, with_loss=True)
        for k in range(3):
            if k == 2:
                g = graph(cell, with_loss=True)
            loss, h, grads = g.grad_trees(dt, dp, rdf.BF16, reproducible=reproducible)
            runs.append((loss.clone(), h.clone(), {n: v.clone() for n, v in grads.items()}))
        spread = {}
        for loss, h, grads in runs[1:]:
            assert torch.equal(h, runs[0][1])
            if reproducible:
                assert torch.equal(loss, runs[0][0])
                for n in grads:
                    assert torch.equal(grads[n], runs[0][2][n]), n
            else:
                assert abs(loss.item() - runs[0][0].item()) <= 1e-6 * abs(runs[0][0].item())
                for n in grads:
                    ref = runs[0][2][n]
                    spread[n] = max(spread.get(n, 0.0), float((grads[n] - ref).abs().max() / ref.abs().max().clamp_min(1e-30)))
        if not reproducible:
            print("run-to-run spread:", spread)
            assert all(v <= 1e-5 for v in spread.values()), spread
    # the reproducible results against the oracle
    want_loss, G, roots = direct.loss_and_grad_pool(tb, p, cell, workers=WORKERS)
    loss, h, grads = runs[0]
    tol = TOL[rdf.BF16]
    assert relerr(h.cpu().numpy(), roots) <= tol and abs(loss.item() - want_loss) <= tol * abs(want_loss)
    errs = {k: relerr(grads[k].cpu().numpy(), G[k]) for k in G}
    assert all(e <= tol for e in errs.values()), errs
    check_embedding_rows(tb, grads["E"].cpu().numpy(), G["E"], tol)
    # reproducible sums exist on the tensor-core path only
    with pytest.raises(rdf.RdfError) as e:
        graph(cell, with_loss=True).grad_trees(dt, dp, rdf.F32, reproducible=True)
    assert e.value.code == -11


def test_depth_stress_config5_forward_sampled():
    """Full config 5 forward (chains of depth 4096, perfect trees of 2^16 leaves); the oracle
    evaluates one chain and one perfect tree."""
    cfg = workloads.config(5)
    st = check_forward(cfg, trees=[0, 63, 64])
    assert st["waves"] >= 2 * 4096


def test_depth_stress_config5_full_size_gradients():
    """Config 5 at full size, forward + backward in fp32: 64 chains of depth 4096 and 16 perfect trees of
    2^16 leaves (2.6 M invocations); every output against the fp64 oracle run over a pool of processes."""
    st, errs = check_grad(workloads.config(5), rdf.F32, workers=WORKERS)
    print("config 5 errors:", errs)
    assert st["waves_backward"] >= 4096
