"""TEST INFRASTRUCTURE (CPU oracle) -- the transformation of Section 3.

Turns a set S of function graphs (one of them named `result`) into one static
graph that uses Call_i / Return_i instead of function-call nodes.  The steps
are those of the general algorithm at the end of Section 3, in its order:

  1. number the n nodes that call f from 0 to n-1;
  2. replace the i-th of them by m nodes Call_i, one per formal parameter,
     each keeping the single input that fed that parameter;
  3. replace the m input nodes of f by Merge nodes fed by the Call_i of the
     matching parameter;
  4. connect f's output to n new nodes Return_0..Return_{n-1}; the output of
     Return_i goes where the output of the i-th call node went;
  5. add a control edge Call_i -> Return_i.

One more kind of edge comes from Figure 3 rather than from the list: inside a
called function every constant gets a control edge from the entry Merge, so
that it emits once per activation (the figure draws Merge -> 1 twice).

Functions with several outputs (the paired function of Section 4 has m + n of
them: the outputs of f and the gradient outputs of f^grad) get one Return_i per
output and call site; output j of call node i feeds the consumers of that
output.  The control edge of step 5 connects the Call_i and Return_i nodes of
the same half (forward or gradient) of such a function.

Readings taken where the text is silent:
  * the numbering order is free (Section 3 says any assignment of the numbers
    works); here call nodes are numbered in the order result-first, then the
    other graphs in the order given, nodes in creation order.  For the
    factorial example this gives Call_0 in `result` and Call_1 in `fact`, as
    in Figure 3.
  * numbering restarts at 0 for every callee f: step 1 numbers the call nodes
    of one f at a time.
"""
from __future__ import annotations

from .graphs import Graph


def transform(functions, result_name: str = "result") -> Graph:
    fs = sorted(functions, key=lambda f: 0 if f.name == result_name else 1)
    assert fs and fs[0].name == result_name, "the program needs a definition of `result`"
    names = {f.name for f in fs}

    # ---- put all graphs side by side in one node space ---------------------
    g = Graph()
    in_of, out_of = {}, {}
    for f in fs:
        off = len(g.nodes)
        for n in f.g.nodes:
            g.add(n.kind, name=n.name, value=n.value, func=n.func, n_in=n.n_in, param=n.param)
        for e in f.g.edges:
            g.connect(e.src + off, e.dst + off, e.dst_port, e.src_port, e.control)
        in_of[f.name] = [i + off for i in f.inputs]
        out_of[f.name] = [o + off for o in f.outs]
    removed = set()

    for f in fs:
        if f.name == result_name:
            continue
        m = f.n_params
        # step 1: number the call nodes of f
        calls = [n.id for n in g.nodes if n.kind == "fcall" and n.name == f.name]
        n_calls = len(calls)
        if n_calls == 0:
            continue
        for c in calls:
            assert g.nodes[c].n_in == m, f"call of {f.name} with wrong arity"
        # step 3 (node part): the input nodes of f become Merge nodes
        entry = []
        for k, nid in enumerate(in_of[f.name]):
            node = g.nodes[nid]
            node.kind, node.name, node.param, node.n_in = "merge", "entry", k, n_calls
            entry.append(nid)
        # the single edge that feeds each output node of f
        out_edges = []
        for o in out_of[f.name]:
            (oe,) = g.in_edges(o)
            out_edges.append(oe)
            removed.add(o)
        for i, c in enumerate(calls):
            # step 2: m nodes Call_i, each with the one input of its parameter
            call_nodes = []
            for k in range(m):
                # (an argument that is itself a call was re-wired to that call's Return_j already)
                (arg_edge,) = [e for e in g.in_edges(c) if e.dst_port == k and e.src not in removed]
                cid = g.add("Call", name=f.name, value=i, func=g.nodes[c].func, n_in=1, param=k)
                g.connect(arg_edge.src, cid, 0, src_port=arg_edge.src_port)
                # step 3 (edge part)
                g.connect(cid, entry[k], i)
                call_nodes.append(cid)
            # step 4: Return_i takes f's output and feeds the old consumers (one Return_i per output)
            consumers = g.out_edges(c)
            for j, out_edge in enumerate(out_edges):
                rid = g.add("Return", name=f.name, value=i, func=g.nodes[c].func, n_in=1, param=j)
                g.connect(out_edge.src, rid, 0, src_port=out_edge.src_port)
                for e in consumers:
                    if e.src_port == j:
                        g.connect(rid, e.dst, e.dst_port, 0, e.control)
                # step 5: control edge(s) Call_i -> Return_i
                for k, cid in enumerate(call_nodes):
                    if (k in f.grad_params) == (j in f.grad_outputs):
                        g.connect(cid, rid, -1, control=True)
            removed.add(c)
        # Figure 3: constants of a called function are triggered by its entry Merge
        for n in g.nodes:
            if n.kind == "const" and n.func == f.name:
                g.connect(entry[0], n.id, -1, control=True)

    for n in g.nodes:
        assert not (n.kind == "fcall" and n.name not in names), f"call of undefined function {n.name}"

    # ---- drop the replaced nodes and renumber -------------------------------
    keep = [n for n in g.nodes if n.id not in removed]
    new_id = {n.id: j for j, n in enumerate(keep)}
    out = Graph()
    for n in keep:
        out.add(n.kind, name=n.name, value=n.value, func=n.func, n_in=n.n_in, param=n.param)
    for e in g.edges:
        if e.src in removed or e.dst in removed:
            continue
        out.connect(new_id[e.src], new_id[e.dst], e.dst_port, e.src_port, e.control)
    return out
