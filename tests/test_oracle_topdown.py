"""Pins for the oracle's top-down (data-dependent) recursion -- Section 6.2, last paragraph: a recursion whose
shape is decided by the values it computes.  `direct.topdown` is the plain recursion; `programs.topdown_program`
is the same definition as a set of function graphs run by the literal tagged-token interpreter after the
transformation of Section 3.  Pinned by: expressions written out by hand for depth limits 0 and 1; closed forms
when the gate never / always stops (a single invocation; the full binary tree with 2^(D+1) - 1 `expand`
invocations); a hand-built 2-dimensional case whose gate stops every left child and expands every right child
(a spine of 2D + 1 `expand` invocations); and the two formulations against each other on random inputs."""
import numpy as np
import pytest

import workloads
from oracle import direct, programs, tagged, transform


def small_params(seed, V=30, H=6, scale=1.0):
    P = workloads.topdown_params(seed, V, H)
    P["E"] = (P["E"] * scale).astype(np.float32)
    return P


def f64(P):
    return {k: np.asarray(v, dtype=np.float64) for k, v in P.items()}


def test_depth_limit_zero_returns_the_seed():
    P = small_params(1)
    for tok in range(5):
        log = {}
        h = direct.topdown(P, tok, 0, log)
        assert np.array_equal(h, f64(P)["E"][tok])
        assert log["expand"] == 1 and log["child"] == 0 and log["margin"] == np.inf


def test_depth_limit_one_written_out():
    P = small_params(2)
    Q = f64(P)
    H = Q["W"].shape[0]
    seen = set()
    for tok in range(30):
        e = Q["E"][tok]
        stops = Q["W_s"][0] @ e + Q["b_s"][0] > 0
        seen.add(bool(stops))
        if stops:
            want = e
        else:
            l = np.tanh(Q["W"][:, :H] @ e + Q["b"])
            r = np.tanh(Q["W"][:, H:] @ e + Q["b"])
            want = np.tanh(Q["W"] @ np.concatenate([l, r]) + Q["b"])      # the children are at the limit: returned as they are
        np.testing.assert_allclose(direct.topdown(P, tok, 1), want, rtol=0, atol=1e-15)
    assert seen == {True, False}                                          # both sides of the gate occur among the seeds


@pytest.mark.parametrize("D", [1, 3, 5])
def test_gate_never_stops_full_tree_closed_form(D):
    P = small_params(3)
    P["b_s"][0] = -100.0                       # gate(h) false for every bounded state
    P["W"][:] = 0.0                            # every child and every cell is tanh(b)
    P["b"] = np.linspace(-1, 1, P["b"].shape[0]).astype(np.float32)
    log = {}
    h = direct.topdown(P, 0, D, log)
    np.testing.assert_allclose(h, np.tanh(P["b"].astype(np.float64)), rtol=0, atol=1e-15)
    assert log["expand"] == 2 ** (D + 1) - 1 and log["child"] == 2 ** (D + 1) - 2


def test_gate_always_stops_single_invocation():
    P = small_params(4)
    P["b_s"][0] = 100.0
    log = {}
    h = direct.topdown(P, 7, 9, log)
    assert np.array_equal(h, f64(P)["E"][7]) and log == {"expand": 1, "child": 0, "margin": log["margin"]}
    assert log["margin"] > 90


def test_spine_shaped_by_the_values():
    """H = 2.  gate(h) = h[0] > 0.  left(h) = tanh((+3, 0)) has a positive first entry: it stops at once;
    right(h) = tanh((-3, 0)): negative, it is expanded again.  So the generated tree is a right spine down to the
    depth limit: D levels with two children each + the seed = 2D + 1 `expand` invocations, whatever D."""
    H = 2
    P = {"E": np.array([[-0.5, 0.25]], dtype=np.float32),
         "W": np.zeros((H, 2 * H), dtype=np.float32),
         "b": np.zeros(H, dtype=np.float32),
         "W_s": np.zeros((5, H), dtype=np.float32), "b_s": np.zeros(5, dtype=np.float32)}
    P["W_s"][0, 0] = 1.0
    # left half: first output = -6 * h[0] (+3 for h[0] = -0.5, and +6 tanh(3) > 0 for h = right(.)); right half: +6 * h[0]
    P["W"][0, 0] = -6.0
    P["W"][0, H + 0] = 6.0
    for D in (1, 2, 4, 7):
        log = {}
        direct.topdown(P, 0, D, log)
        assert log["expand"] == 2 * D + 1 and log["child"] == 2 * D, (D, log)
    # and the value for D = 1 by hand: cell(left, right) with left = tanh(3, 0), right = tanh(-3, 0)
    l, r = np.tanh([3.0, 0.0]), np.tanh([-3.0, 0.0])
    want = np.tanh(P["W"].astype(np.float64) @ np.concatenate([l, r]))
    np.testing.assert_allclose(direct.topdown(P, 0, 1), want, rtol=0, atol=1e-15)


@pytest.mark.parametrize("dead", [True, False])
def test_tagged_interpreter_runs_the_same_recursion(dead):
    V, H, D = 40, 6, 5
    P = small_params(5, V, H)
    tb = workloads.topdown_batch(5, 12, V)
    g = transform.transform(programs.topdown_program())
    ops = programs.topdown_ops(tb, P, D)
    fired = {"gate": 0, "child_l": 0, "child_r": 0, "cell_rnn": 0}

    def counted(name, fn):
        def run_op(*a):
            fired[name] += 1
            return fn(*a)
        return run_op

    for name in fired:
        ops[name] = counted(name, ops[name])
    sizes = set()
    for b in range(tb.B):
        log = {}
        want = direct.topdown(P, int(tb.tok[b]), D, log)
        r = tagged.run(g, {0: int(tb.tree_root[b])}, ops, dead_tokens=dead)
        np.testing.assert_allclose(r.value, want, rtol=0, atol=1e-14)
        assert r.leftover == 0
        # the gate fires once per `expand` invocation, a child operator once per `left` / `right` invocation, and
        # every expanded node ends in one cell
        assert fired == {"gate": log["expand"], "child_l": log["child"] // 2, "child_r": log["child"] // 2,
                         "cell_rnn": log["child"] // 2}
        fired.update(dict.fromkeys(fired, 0))
        sizes.add(log["expand"])
    assert len(sizes) >= 4                     # the seeds generate trees of different sizes


def test_workload_recipe_generates_a_spread_of_tree_sizes():
    P = workloads.topdown_params(workloads.DEFAULT_SEED, 1000, 64)
    tb = workloads.topdown_batch(workloads.DEFAULT_SEED, 128, 1000)
    assert tb.N == tb.B == 128 and (tb.left < 0).all()
    sizes = []
    for b in range(tb.B):
        log = {}
        direct.topdown(P, int(tb.tok[b]), 8, log)
        sizes.append(log["expand"])
    sizes = np.array(sizes)
    assert sizes.min() == 1 and sizes.max() > 50 and 1 < np.median(sizes) < 20
