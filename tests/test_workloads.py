"""Pins of the seeded input generators (CPU): the parity of the bf16 workloads rests on `bf16_round`, and the
benchmark's invocation counts on the tree generators, so both are checked against something other than
themselves: torch's own fp32 -> bf16 conversion, the size formulas of full binary trees, and the stated
shape of every workload (clip range and median of the leaf counts, chain and perfect-tree sizes)."""
import numpy as np
import pytest

import workloads
from workloads import gen

torch = pytest.importorskip("torch")


def test_bf16_round_is_round_to_nearest_even():
    rng = np.random.default_rng(5)
    x = np.concatenate([
        rng.standard_normal(20000).astype(np.float32) * np.float32(10.0) ** rng.integers(-20, 20, 20000).astype(np.float32),
        np.array([0.0, -0.0, 1.0, -1.0, 3.0e38, -3.0e38, 1e-40, -1e-40], dtype=np.float32),
    ])
    # exact ties between two bf16 neighbours: mantissa bits 0x8000 below an even and below an odd bf16 value
    ties = np.array([0x3F808000, 0x3F818000, 0xBF808000, 0xBF818000, 0x00008000, 0x00018000, 0x7F7E8000],
                    dtype=np.uint32).view(np.float32)
    x = np.concatenate([x, ties])
    want = torch.from_numpy(x).bfloat16().float().numpy()
    got = workloads.bf16_round(x)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    assert got[-7:].view(np.uint32).tolist() == [0x3F800000, 0x3F820000, 0xBF800000, 0xBF820000, 0x00000000, 0x00020000,
                                                 0x7F7E0000]        # ties go to the even neighbour
    assert np.array_equal(workloads.bf16_round(got), got)             # idempotent


def _leaf_counts(tb):
    leaves = np.zeros(tb.B, dtype=np.int64)
    sizes = tb.tree_sizes()
    for t in range(tb.B):
        s = int(tb.tree_root[t])
        leaves[t] = int((tb.left[s:s + int(sizes[t])] < 0).sum())
    return leaves, sizes


def test_config3_tree_sizes():
    cfg = workloads.config(3)
    tb = cfg["trees"]
    L, sizes = _leaf_counts(tb)
    assert tb.B == 8192 and L.min() >= 1 and L.max() == 56          # clipped to [1, 56]; the clip is reached
    assert np.median(L) == 18                                        # the stated median
    assert np.array_equal(sizes, 2 * L - 1)                          # full binary trees: 2L - 1 nodes
    assert tb.N == int((2 * L - 1).sum()) == 323816                  # the benchmark's invocation count (default seed)
    assert tb.n_cells == int((L - 1).sum()) == 157812
    assert 19.5 < L.mean() < 21.0                                    # lognormal(ln 18, 0.5): mean about 20.3
    # every internal node has two children inside its own tree, every leaf a token below the vocabulary
    internal = tb.left >= 0
    assert np.all((tb.right >= 0) == internal)
    assert np.all(tb.tok[~internal] >= 0) and tb.tok.max() < cfg["V"] and np.all(tb.tok[internal] == -1)
    assert tb.label.min() == 0 and tb.label.max() == 4
    # config 4 draws the same trees
    tb4 = workloads.config(4)["trees"]
    assert np.array_equal(tb4.left, tb.left) and np.array_equal(tb4.tok, tb.tok)
    # parameters of the bf16 workloads are bf16-representable
    for v in cfg["params"].values():
        assert np.array_equal(workloads.bf16_round(v), v)


def test_config2_and_config1_shapes():
    tb = workloads.config(2)["trees"]
    L, sizes = _leaf_counts(tb)
    assert tb.B == 512 and L.min() >= 2 and L.max() <= 32 and np.array_equal(sizes, 2 * L - 1)
    x = workloads.config(1)["x"]
    assert x.shape == (1024,) and x.min() == 0 and x.max() == 18 and x.dtype == np.int64


def test_config5_sizes():
    tb = workloads.config(5)["trees"]
    assert tb.B == 80
    assert tb.N == 64 * 8193 + 16 * 131071 == 2621488
    assert tb.n_cells == 64 * 4096 + 16 * 65535 == 1310704
    sizes = tb.tree_sizes()
    assert sizes[:64].tolist() == [8193] * 64 and sizes[64:].tolist() == [131071] * 16
    # a chain: every right child is a leaf, the left child continues
    l, r = gen.chain_tree_shape(4096)
    internal = np.flatnonzero(l >= 0)
    assert len(internal) == 4096 and np.all(l[r[internal]] < 0)
    depth, v = 0, 0
    while l[v] >= 0:
        v, depth = int(l[v]), depth + 1
    assert depth == 4096


def test_random_split_is_a_full_binary_tree_and_seeded():
    rng = np.random.default_rng(1)
    for L in (1, 2, 3, 17, 56):
        l, r = workloads.random_split_shape(rng, L)
        assert len(l) == 2 * L - 1 and int((l < 0).sum()) == L
        seen = np.zeros(len(l), dtype=int)                           # every node but the root is one node's child
        for a in np.concatenate([l[l >= 0], r[r >= 0]]):
            seen[a] += 1
        assert seen[0] == 0 and np.all(seen[1:] == 1)
    a, b = workloads.config(3, B=50)["trees"], workloads.config(3, B=50)["trees"]
    assert np.array_equal(a.left, b.left) and np.array_equal(a.label, b.label)
    c = workloads.config(3, B=50, seed=7)["trees"]
    assert c.N != a.N or not np.array_equal(c.left, a.left)
