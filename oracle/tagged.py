"""TEST INFRASTRUCTURE (CPU oracle) -- a literal tagged-token interpreter.

Executes the single static graph produced by `transform.py`, one token at a
time, following the paper's semantic equations:

  * a token is a pair <tag, datum>; a tag is a list of labels, head first
    (footnote on the (n:t) notation, Section 2.3);
  * a processing node fires when all its inputs hold tokens with exactly the
    same tag and emits a token with that tag (Section 2.2);
  * `*` ("hiaton", a dead datum) is propagated by every operator except Merge;
    Switch(true, d) = (d, *), Switch(false, d) = (*, d); Merge forwards the
    input that is not a hiaton (Section 2.2);
  * Call_i <t, d> = <i:t, d>;  Return_i <i:t, d> = <t, d>  (Section 3);
  * Return_i offered a token whose tag does not start with i emits nothing
    (Section 5.1: the frame's label is checked first);
  * a hiaton reaching Call_i does not enter the function body: it travels
    along the control edge Call_i -> Return_i, and Return_i hands it on to its
    successors (Section 5.2.1);
  * nodes wait in a pending table keyed by (node, tag) and tokens are taken
    from a FIFO queue until it is empty (Section 5.1);
  * Enter <t, d> = <0:t, d>;  Exit <n:t, d> = <t, d>;  Next <n:t, d> = <(n+1):t, d>
    (Section 2.3).  Iteration counters and call labels live in the one tag list
    (Section 5.1: loops and functions share the stack).

Readings where the text is silent:
  * the entry Merge of a function has one input per call site; tokens from
    different call sites carry different tags, so at most one live token per
    tag ever arrives and it is forwarded as it arrives;
  * a constant inside a called function fires when the control token from the
    entry Merge arrives (Figure 3); a constant of `result` fires once, with
    the empty tag;
  * a hiaton that reaches Exit or Next is dropped: every iteration but the last sends one to Exit (the Switch's
    other side) and the last one sends one round the body to Next; letting them through would put several tokens
    with one tag on the loop's consumers, or keep a dead loop turning (the paper does not treat this case);
  * `dead_tokens=False` elides hiatons altogether (Switch emits only the live
    side).  Results are the same; operands left waiting for a partner on the
    branch not taken are dropped when the queue runs empty.

Only tests, the smoke check and the CPU-baseline leg of the benchmark may
import anything under `oracle/`.
"""
from __future__ import annotations

from collections import deque


class _Hiaton:
    def __repr__(self):
        return "*"


DEAD = _Hiaton()


class RunResult:
    def __init__(self):
        self.outputs = {}        # tag -> datum, tokens that reached the output node
        self.calls = {}          # tag after the push (tuple) -> argument datum(s) by parameter
        self.returns = {}        # tag before the pop (tuple) -> returned datum (output 0 of the function)
        self.returns_by_output = {}   # (tag, output index) -> returned datum, for functions with several outputs
        self.firings = 0
        self.max_depth = 0
        self.enters = []         # tags produced by Enter nodes, in firing order
        self.nexts = []          # tags produced by Next nodes
        self.exits = []          # tags consumed by Exit nodes
        self.leftover = 0        # tokens still waiting when the queue ran empty
        self.max_pending = 0

    @property
    def value(self):
        return self.outputs[()]


def run(graph, feeds, ops, dead_tokens=True, max_firings=None) -> RunResult:
    """Run `graph` on one instance.

    feeds: {parameter index of `result`: datum}; ops: {symbol: python callable}.
    """
    nodes = graph.nodes
    outs = [[] for _ in nodes]          # per node: (src_port, dst, dst_port)
    has_ctrl_in = [False] * len(nodes)
    for e in graph.edges:
        outs[e.src].append((e.src_port, e.dst, -1 if e.control else e.dst_port))
        if e.control:
            has_ctrl_in[e.dst] = True

    res = RunResult()
    queue = deque()
    pending = {}                         # (node, tag) -> {port: datum}
    ctrl = {}                            # (Return node, tag) -> live control token waiting
    held = {}                            # (Return node, tag) -> output datum waiting for it

    def emit(nid, port, tag, datum):
        for sp, dst, dp in outs[nid]:
            if sp == port:
                queue.append((dst, dp, tag, datum))

    # input nodes of `result` and its constants start the run with the empty tag
    for n in nodes:
        if n.kind == "in":
            emit(n.id, 0, (), feeds[n.value])
        elif n.kind == "const" and not has_ctrl_in[n.id]:
            emit(n.id, 0, (), n.value)

    while queue:
        nid, port, tag, datum = queue.popleft()
        n = nodes[nid]
        kind = n.kind
        res.firings += 1
        if max_firings is not None and res.firings > max_firings:
            raise RuntimeError("firing limit exceeded (non-terminating recursion?)")

        if kind == "op" or kind == "switch":
            if n.n_in > 1:
                key = (nid, tag)
                slot = pending.setdefault(key, {})
                assert port not in slot, "two tokens with one tag on one input"
                slot[port] = datum
                if len(pending) > res.max_pending:
                    res.max_pending = len(pending)
                if len(slot) < n.n_in:
                    continue
                del pending[key]
                args = [slot[p] for p in range(n.n_in)]
            else:
                args = [datum]
            dead = any(a is DEAD for a in args)
            if kind == "op":
                emit(nid, 0, tag, DEAD if dead else ops[n.name](*args))
            else:
                pred, d = args
                if dead:
                    live_t = live_f = DEAD
                elif pred:
                    live_t, live_f = d, DEAD
                else:
                    live_t, live_f = DEAD, d
                if dead_tokens or live_t is not DEAD:
                    emit(nid, 0, tag, live_t)
                if dead_tokens or live_f is not DEAD:
                    emit(nid, 1, tag, live_f)
        elif kind == "const":
            assert port == -1
            emit(nid, 0, tag, n.value)
        elif kind == "merge":
            if datum is not DEAD:
                emit(nid, 0, tag, datum)
        elif kind == "Call":
            new_tag = (n.value,) + tag
            if datum is DEAD:
                # only the control edge carries it on (to Return_i)
                for sp, dst, dp in outs[nid]:
                    if dp == -1:
                        queue.append((dst, -1, new_tag, DEAD))
            else:
                res.calls.setdefault(new_tag, {})[n.param] = datum
                if len(new_tag) > res.max_depth:
                    res.max_depth = len(new_tag)
                for sp, dst, dp in outs[nid]:
                    queue.append((dst, dp, new_tag, datum))
        elif kind == "Return":
            # two inputs with the same tag: the control token of Call_i and the
            # function's output; either may come first
            key = (nid, tag)
            if port == -1:
                if datum is DEAD:
                    emit(nid, 0, tag[1:], DEAD)
                elif key in held:
                    d = held.pop(key)
                    res.returns_by_output[(tag, n.param)] = d
                    if n.param == 0:
                        res.returns[tag] = d
                    emit(nid, 0, tag[1:], d)
                else:
                    ctrl[key] = True
            else:
                if datum is DEAD:
                    continue
                if not tag or tag[0] != n.value:
                    continue                      # label mismatch: no output
                if ctrl.pop(key, False):
                    res.returns_by_output[(tag, n.param)] = datum
                    if n.param == 0:
                        res.returns[tag] = datum
                    emit(nid, 0, tag[1:], datum)
                else:
                    held[key] = datum
        elif kind == "Enter":
            if datum is not DEAD:
                res.enters.append((0,) + tag)
                if len(tag) + 1 > res.max_depth:
                    res.max_depth = len(tag) + 1
            emit(nid, 0, (0,) + tag, datum)
        elif kind == "Exit":
            if datum is not DEAD:
                res.exits.append(tag)
                emit(nid, 0, tag[1:], datum)
        elif kind == "Next":
            if datum is not DEAD:
                res.nexts.append((tag[0] + 1,) + tag[1:])
                emit(nid, 0, (tag[0] + 1,) + tag[1:], datum)
        elif kind == "out":
            if datum is not DEAD:
                assert tag not in res.outputs
                res.outputs[tag] = datum
        else:
            raise AssertionError(f"node kind {kind} cannot receive tokens")

    res.leftover = sum(len(s) for s in pending.values()) + len(ctrl) + len(held)
    return res
