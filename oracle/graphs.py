"""TEST INFRASTRUCTURE (CPU oracle) -- dataflow graphs as plain node/edge lists.

A dataflow graph is a directed graph whose nodes are input nodes, output
nodes and processing nodes (Definition 1, Section 2.1).  A program is a *set*
of such graphs, one per function, in which a node may carry the name of a
defined function (Section 2.4, Figure 2).  This module only holds the data
structure and a small builder; the transformation to a single static graph is
in `transform.py`, execution in `tagged.py`.

Only tests, the smoke check and the CPU-baseline leg of the benchmark may
import anything under `oracle/`.
"""
from __future__ import annotations

from dataclasses import dataclass, field


@dataclass
class Node:
    id: int
    kind: str            # 'in' 'out' 'const' 'op' 'switch' 'merge' 'fcall' 'Call' 'Return'
    name: str = ""       # op symbol, or callee name for 'fcall', or owner function
    value: object = None  # constant value / parameter index / label i
    func: str = ""       # the function graph this node came from
    n_in: int = 0        # number of data input ports
    param: int = 0       # for 'Call'/'merge' made from parameter k: k; for 'Return'/'out' of output j: j


@dataclass
class Edge:
    src: int
    src_port: int        # Switch: 0 = true output, 1 = false output
    dst: int
    dst_port: int        # data input port; -1 for a control edge
    control: bool = False


@dataclass
class Graph:
    nodes: list = field(default_factory=list)
    edges: list = field(default_factory=list)

    def add(self, kind, **kw) -> int:
        n = Node(id=len(self.nodes), kind=kind, **kw)
        self.nodes.append(n)
        return n.id

    def connect(self, src, dst, dst_port, src_port=0, control=False):
        self.edges.append(Edge(src, src_port, dst, dst_port, control))

    def out_edges(self, nid):
        return [e for e in self.edges if e.src == nid]

    def in_edges(self, nid):
        return [e for e in self.edges if e.dst == nid]

    def count(self, kind, name=None):
        return sum(1 for n in self.nodes if n.kind == kind and (name is None or n.name == name))


class FunctionGraph:
    """Builder for the graph of one function (Figure 2 style).

    Values handed around while building are (node id, output port) pairs.
    """

    def __init__(self, name: str, n_params: int):
        self.name = name
        self.n_params = n_params
        self.g = Graph()
        self.inputs = [self.g.add("in", value=k, func=name) for k in range(n_params)]
        self.out = None          # the output node (the first one of a function with several outputs)
        self.outs = []           # all output nodes, in order
        # For a function that pairs a forward computation with its gradient computation (Section 4): which
        # parameters and which outputs belong to the gradient half.  The control edge Call_i -> Return_i is
        # drawn between nodes of the same half only (the forward Return_i must not wait for the gradient
        # Call_i, which fires in the backward phase).
        self.grad_params = set()
        self.grad_outputs = set()

    def param(self, k=0):
        return (self.inputs[k], 0)

    def const(self, v):
        return (self.g.add("const", value=v, func=self.name), 0)

    def op(self, sym, *args):
        nid = self.g.add("op", name=sym, func=self.name, n_in=len(args))
        for p, (s, sp) in enumerate(args):
            self.g.connect(s, nid, p, src_port=sp)
        return (nid, 0)

    def switch(self, pred, data):
        """Returns (true output, false output)."""
        nid = self.g.add("switch", func=self.name, n_in=2)
        self.g.connect(pred[0], nid, 0, src_port=pred[1])
        self.g.connect(data[0], nid, 1, src_port=data[1])
        return (nid, 0), (nid, 1)

    def merge(self, a, b):
        nid = self.g.add("merge", func=self.name, n_in=2)
        self.g.connect(a[0], nid, 0, src_port=a[1])
        self.g.connect(b[0], nid, 1, src_port=b[1])
        return (nid, 0)

    def call(self, fname, *args):
        nid = self.g.add("fcall", name=fname, func=self.name, n_in=len(args))
        for p, (s, sp) in enumerate(args):
            self.g.connect(s, nid, p, src_port=sp)
        return (nid, 0)

    def call_open(self, fname, n_args):
        """A call node whose arguments are connected afterwards with `set_arg` (needed where an argument
        depends on one of the call's own outputs, as the gradient input of a paired call does).
        Output j of the callee is the value (node, j)."""
        return self.g.add("fcall", name=fname, func=self.name, n_in=n_args)

    def set_arg(self, call_node, port, v):
        self.g.connect(v[0], call_node, port, src_port=v[1])

    def output(self, v):
        nid = self.g.add("out", func=self.name, n_in=1, param=len(self.outs))
        self.g.connect(v[0], nid, 0, src_port=v[1])
        self.outs.append(nid)
        if self.out is None:
            self.out = nid
        return nid
