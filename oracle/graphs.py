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
    kind: str            # 'in' 'out' 'const' 'op' 'switch' 'merge' 'fcall' 'Call' 'Return' 'Enter' 'Exit' 'Next'
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

    # ---- tagged iteration (Section 2.3, the while-loop of Figure 1)
    def enter(self, v):
        nid = self.g.add("Enter", func=self.name, n_in=1)
        self.g.connect(v[0], nid, 0, src_port=v[1])
        return (nid, 0)

    def exit_(self, v):
        nid = self.g.add("Exit", func=self.name, n_in=1)
        self.g.connect(v[0], nid, 0, src_port=v[1])
        return (nid, 0)

    def next_(self, v):
        nid = self.g.add("Next", func=self.name, n_in=1)
        self.g.connect(v[0], nid, 0, src_port=v[1])
        return (nid, 0)

    def loop_merge(self, entered):
        """The Merge at the head of a loop: input 0 from Enter now, input 1 from Next through `close_loop`."""
        nid = self.g.add("merge", name="loop", func=self.name, n_in=2)
        self.g.connect(entered[0], nid, 0, src_port=entered[1])
        return (nid, 0)

    def close_loop(self, merge, nxt):
        self.g.connect(nxt[0], merge[0], 1, src_port=nxt[1])

    def while_loop(self, inits, cond, body, result):
        """The graph of Figure 1 for loop-carried variables v_1..v_m, one Enter / Merge / Switch / Next per variable
        and an Exit for the variable that is the loop's value:
            inits  : initial values (outside the loop);
            cond   : f(builder, merged values) -> predicate value;
            body   : f(builder, values on the true side) -> next values;
            result : index of the variable whose final value leaves through Exit.
        Inside `cond` and `body` constants must be derived from a loop value with a unary operator (a constant node
        would carry the tag of the enclosing activation, not of the iteration)."""
        merged = [self.loop_merge(self.enter(v)) for v in inits]
        p = cond(self, merged)
        sides = [self.switch(p, m) for m in merged]
        nxt = body(self, [t for t, _ in sides])
        assert len(nxt) == len(inits)
        for m, n in zip(merged, nxt):
            self.close_loop(m, self.next_(n))
        return self.exit_(sides[result][1])

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
