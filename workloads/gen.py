"""Seeded generators for the five benchmark workloads.

Shapes, sizes and value distributions follow the workload list the build is
measured on (recursive Fibonacci calls; random binary trees with per-node
labels standing in for a sentiment treebank; a depth stress mix of degenerate
chains and perfect trees).  Everything here is input drawing: no tags, no
cells, no gradients.

Tree container (flat arrays over the whole batch, int32):
    tree_root[B]  global index of each tree's root node
    left[N], right[N]  global child indices, -1 at leaves (full binary trees)
    tok[N]   token id at leaves, -1 at internal nodes
    label[N] class label of every node (leaves and internal)
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

DEFAULT_SEED = 20241028


# --------------------------------------------------------------------------
# helpers
# --------------------------------------------------------------------------
def _rng(seed: int, stream: int) -> np.random.Generator:
    """Independent deterministic streams: one per kind of input."""
    return np.random.Generator(np.random.PCG64([int(seed), int(stream)]))


def bf16_round(x: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bfloat16 (ties to even) and return them
    widened back to fp32.  Used once on parameters of the bf16 workloads so
    that every consumer starts from the same representable values."""
    a = np.ascontiguousarray(x, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    u = (u + 0x7FFF + lsb) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(a.shape)


# --------------------------------------------------------------------------
# workload 1: integer recursion
# --------------------------------------------------------------------------
def fib_batch(seed: int = DEFAULT_SEED, B: int = 1024, n_lo: int = 0, n_hi: int = 18) -> np.ndarray:
    """B independent arguments n ~ U{n_lo..n_hi}, int64."""
    return _rng(seed, 1).integers(n_lo, n_hi + 1, size=B, dtype=np.int64)


# --------------------------------------------------------------------------
# tree shapes (local numbering, root = 0)
# --------------------------------------------------------------------------
def random_split_shape(rng: np.random.Generator, L: int):
    """Full binary tree with L leaves: a node with l > 1 leaves below it draws
    k ~ U{1..l-1} and gives k leaves to its left child, l-k to its right.
    Nodes are numbered in pre-order.  Returns (left, right) as int32 arrays."""
    n = 2 * L - 1
    left = np.full(n, -1, dtype=np.int32)
    right = np.full(n, -1, dtype=np.int32)
    stack = [(0, L)]
    while stack:
        node, l = stack.pop()
        if l == 1:
            continue
        k = int(rng.integers(1, l))
        # pre-order: the left subtree (2k-1 nodes) follows its parent directly
        left[node] = node + 1
        right[node] = node + 2 * k
        stack.append((node + 2 * k, l - k))
        stack.append((node + 1, k))
    return left, right


def chain_tree_shape(depth: int):
    """Left-degenerate chain: `depth` internal nodes, each with a leaf as right
    child; the left child continues the chain and the last one is a leaf.
    Height = depth, leaves = depth + 1, nodes = 2*depth + 1."""
    n = 2 * depth + 1
    left = np.full(n, -1, dtype=np.int32)
    right = np.full(n, -1, dtype=np.int32)
    i = np.arange(depth, dtype=np.int32)
    left[2 * i] = 2 * i + 2
    right[2 * i] = 2 * i + 1
    return left, right


def perfect_tree_shape(height: int):
    """Perfect binary tree with 2**height leaves in heap numbering."""
    n = 2 ** (height + 1) - 1
    n_int = 2 ** height - 1
    left = np.full(n, -1, dtype=np.int32)
    right = np.full(n, -1, dtype=np.int32)
    i = np.arange(n_int, dtype=np.int32)
    left[i] = 2 * i + 1
    right[i] = 2 * i + 2
    return left, right


# --------------------------------------------------------------------------
# tree batches
# --------------------------------------------------------------------------
@dataclass
class TreeBatch:
    tree_root: np.ndarray  # int32 [B]
    left: np.ndarray       # int32 [N]
    right: np.ndarray      # int32 [N]
    tok: np.ndarray        # int32 [N]
    label: np.ndarray      # int32 [N]

    @property
    def B(self) -> int:
        return int(self.tree_root.shape[0])

    @property
    def N(self) -> int:
        return int(self.left.shape[0])

    @property
    def n_cells(self) -> int:
        return int((self.left >= 0).sum())

    def tree_sizes(self) -> np.ndarray:
        """Nodes per tree (trees are stored contiguously, root first)."""
        ends = np.append(self.tree_root[1:], self.N)
        return (ends - self.tree_root).astype(np.int64)


def tree_batch_from_shapes(shapes, seed: int, vocab: int, n_classes: int = 5) -> TreeBatch:
    """Concatenate local shapes into one flat batch and draw leaf token ids
    ~ U{0..vocab-1} and per-node labels ~ U{0..n_classes-1}."""
    sizes = np.array([s[0].shape[0] for s in shapes], dtype=np.int64)
    offs = np.concatenate([[0], np.cumsum(sizes)[:-1]]).astype(np.int64)
    N = int(sizes.sum())
    left = np.empty(N, dtype=np.int32)
    right = np.empty(N, dtype=np.int32)
    for (l, r), o in zip(shapes, offs):
        n = l.shape[0]
        left[o:o + n] = np.where(l >= 0, l + o, -1)
        right[o:o + n] = np.where(r >= 0, r + o, -1)
    is_leaf = left < 0
    tok = np.full(N, -1, dtype=np.int32)
    tok[is_leaf] = _rng(seed, 3).integers(0, vocab, size=int(is_leaf.sum()), dtype=np.int32)
    label = _rng(seed, 4).integers(0, n_classes, size=N, dtype=np.int32)
    return TreeBatch(offs.astype(np.int32), left, right, tok, label)


def subset_trees(tb: TreeBatch, idx) -> TreeBatch:
    """The trees `idx` (in that order) as a batch of their own, renumbered."""
    sizes = tb.tree_sizes()
    parts = []
    o = 0
    roots = []
    for t in idx:
        s = int(tb.tree_root[t])
        n = int(sizes[t])
        sl = slice(s, s + n)
        shift = o - s
        parts.append((np.where(tb.left[sl] >= 0, tb.left[sl] + shift, -1),
                      np.where(tb.right[sl] >= 0, tb.right[sl] + shift, -1),
                      tb.tok[sl], tb.label[sl]))
        roots.append(o)
        o += n
    cat = lambda k: np.concatenate([p[k] for p in parts]).astype(np.int32)  # noqa: E731
    return TreeBatch(np.array(roots, dtype=np.int32), cat(0), cat(1), cat(2), cat(3))


# --------------------------------------------------------------------------
# parameters
# --------------------------------------------------------------------------
def _xavier(rng, rows, cols):
    a = np.sqrt(6.0 / (rows + cols))
    return rng.uniform(-a, a, size=(rows, cols)).astype(np.float32)


def treernn_params(seed: int, V: int, D: int, H: int, n_classes: int = 5, bf16: bool = False):
    """E [V,D] ~ N(0, 0.1^2); W [H,2H] and W_s [n_classes,H] Xavier-uniform;
    biases zero.  D must equal H (a leaf's state is its embedding row)."""
    assert D == H
    r = _rng(seed, 5)
    p = {
        "E": (0.1 * r.standard_normal((V, D))).astype(np.float32),
        "W": _xavier(r, H, 2 * H),
        "b": np.zeros(H, dtype=np.float32),
        "W_s": _xavier(r, n_classes, H),
        "b_s": np.zeros(n_classes, dtype=np.float32),
    }
    if bf16:
        p = {k: bf16_round(v) for k, v in p.items()}
    return p


def treelstm_params(seed: int, V: int, D: int, H: int, n_classes: int = 5, bf16: bool = False):
    """Binary TreeLSTM: W [5H,2H] (row blocks i, f_l, f_r, o, u), leaf
    projection W_x [3H,D] (row blocks i, o, u), W_s [n_classes,H]; biases 0."""
    r = _rng(seed, 6)
    p = {
        "E": (0.1 * r.standard_normal((V, D))).astype(np.float32),
        "W": _xavier(r, 5 * H, 2 * H),
        "b": np.zeros(5 * H, dtype=np.float32),
        "W_x": _xavier(r, 3 * H, D),
        "b_x": np.zeros(3 * H, dtype=np.float32),
        "W_s": _xavier(r, n_classes, H),
        "b_s": np.zeros(n_classes, dtype=np.float32),
    }
    if bf16:
        p = {k: bf16_round(v) for k, v in p.items()}
    return p


def topdown_params(seed: int, V: int, H: int, stop_bias: float = -0.3):
    """Parameters for the top-down recursion (a tree grown from a seed vector; a gate on the state decides at
    every node whether it is expanded): the TreeRNN parameter set with a seed table E ~ N(0, 1), W scaled by 2 so
    that the child states keep their spread from level to level, and b_s[0] = stop_bias so that a node is expanded
    a little more often than not (the generated trees neither die out at once nor fill every level)."""
    r = _rng(seed, 7)
    return {
        "E": r.standard_normal((V, H)).astype(np.float32),
        "W": (2.0 * _xavier(r, H, 2 * H)).astype(np.float32),
        "b": np.zeros(H, dtype=np.float32),
        "W_s": _xavier(r, 5, H),
        "b_s": np.array([stop_bias, 0, 0, 0, 0], dtype=np.float32),
    }


def topdown_batch(seed: int, B: int, V: int) -> TreeBatch:
    """B seeds: single-node trees whose token selects the seed row."""
    one = (np.full(1, -1, dtype=np.int32), np.full(1, -1, dtype=np.int32))
    return tree_batch_from_shapes([one] * B, seed, vocab=V)


# --------------------------------------------------------------------------
# the five named workloads
# --------------------------------------------------------------------------
def _lognormal_leaves(rng, B, median=18.0, sigma=0.5, lo=1, hi=56):
    L = np.rint(np.exp(rng.normal(np.log(median), sigma, size=B)))
    return np.clip(L, lo, hi).astype(np.int64)


def config(k: int, seed: int = DEFAULT_SEED, B: int | None = None, **over):
    """Workload k (1..5, and 6: the top-down recursion) as a dict.  `B` overrides the batch size (for small
    parity cases); for k == 5 `chains`, `chain_depth`, `perfect`,
    `perfect_height` may be overridden through keyword arguments."""
    if k == 1:
        B = 1024 if B is None else B
        return {"kind": "fib", "x": fib_batch(seed, B, 0, over.get("n_hi", 18)), "B": B}
    if k == 2:
        B = 512 if B is None else B
        r = _rng(seed, 2)
        Ls = r.integers(2, 33, size=B)
        shapes = [random_split_shape(r, int(L)) for L in Ls]
        tb = tree_batch_from_shapes(shapes, seed, vocab=1000)
        return {"kind": "treernn", "trees": tb, "H": 64, "V": 1000, "bf16": False, "grad": False,
                "params": treernn_params(seed, 1000, 64, 64)}
    if k in (3, 4):
        B = 8192 if B is None else B
        r = _rng(seed, 2)
        Ls = _lognormal_leaves(r, B)
        shapes = [random_split_shape(r, int(L)) for L in Ls]
        V, H = over.get("V", 21000), over.get("H", 300)
        tb = tree_batch_from_shapes(shapes, seed, vocab=V)
        if k == 3:
            return {"kind": "treernn", "trees": tb, "H": H, "V": V, "bf16": True, "grad": True,
                    "params": treernn_params(seed, V, H, H, bf16=True)}
        return {"kind": "treelstm", "trees": tb, "H": H, "V": V, "bf16": True, "grad": True,
                "params": treelstm_params(seed, V, H, H, bf16=True)}
    if k == 5:
        chains = over.get("chains", 64)
        depth = over.get("chain_depth", 4096)
        perfect = over.get("perfect", 16)
        height = over.get("perfect_height", 16)
        V, H = over.get("V", 50000), over.get("H", 256)
        shapes = [chain_tree_shape(depth)] * chains + [perfect_tree_shape(height)] * perfect
        tb = tree_batch_from_shapes(shapes, seed, vocab=V)
        return {"kind": "treernn", "trees": tb, "H": H, "V": V, "bf16": False, "grad": True,
                "params": treernn_params(seed, V, H, H)}
    if k == 6:
        # beyond the five named configurations: recursion whose shape follows the values (a tree grown top-down from
        # a seed state, a gate on every node's state deciding whether it is expanded; depth limit D)
        B = 8192 if B is None else B
        V, H, D = over.get("V", 21000), over.get("H", 128), over.get("D", 10)
        return {"kind": "topdown", "trees": topdown_batch(seed, B, V), "H": H, "V": V, "D": D, "bf16": False, "grad": False,
                "params": topdown_params(seed, V, H), "max_invocations": 256 * B}
    raise ValueError(f"unknown workload {k}")
