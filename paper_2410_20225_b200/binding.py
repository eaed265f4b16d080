"""ctypes binding of the C boundary declared in include/rdf.h.

Argument marshalling only: every step of the path (tag push/pop, token
matching, wave scheduling, cells, gradients) runs in the CUDA library.  torch
is used for device memory and streams.  There is no CPU fallback: a missing
library or a missing GPU is an error.
"""
from __future__ import annotations

import ctypes as C

import numpy as np

from . import build as _build

# ---------------------------------------------------------------- constants
RDF_OK = 0
ERRORS = {
    -1: "RDF_ERR_BAD_PROGRAM", -2: "RDF_ERR_BAD_ARG", -3: "RDF_ERR_WORKSPACE_TOO_SMALL", -4: "RDF_ERR_TAG_OVERFLOW",
    -5: "RDF_ERR_STORE_FULL", -6: "RDF_ERR_FRAMES_FULL", -7: "RDF_ERR_QUEUE_FULL", -8: "RDF_ERR_WAVE_LIMIT",
    -9: "RDF_ERR_TIMEOUT", -10: "RDF_ERR_CUDA", -11: "RDF_ERR_UNSUPPORTED",
}
(OP_PARAM, OP_CONST, OP_ADD, OP_SUB, OP_MUL, OP_MAX, OP_LT, OP_EQ, OP_IF, OP_CALL, OP_IS_LEAF, OP_LEFT, OP_RIGHT,
 OP_TOK, OP_EMBED, OP_CELL_RNN, OP_LEAF_LSTM, OP_CELL_LSTM, OP_NODE_LOSS, OP_REM, OP_CHILD_L, OP_CHILD_R,
 OP_GATE) = range(23)
TAGS_PATH, TAGS_FRAME = 0, 1
F32, BF16 = 0, 1
(NODE_IN, NODE_OUT, NODE_CONST, NODE_OP, NODE_SWITCH, NODE_MERGE, NODE_ENTRY_MERGE, NODE_CALL, NODE_RETURN, NODE_ENTER,
 NODE_EXIT, NODE_NEXT) = range(12)
FN_FUNCTION, FN_LOOP = 0, 1
LOOP_LABEL = 255

PATH_BITS, DEPTH_SHIFT, INST_SHIFT = 38, 38, 44


class RdfError(RuntimeError):
    def __init__(self, code, where=""):
        self.code = code
        super().__init__(f"{where}: {ERRORS.get(code, code)}")


# ------------------------------------------------------------------ structs
class rdf_expr(C.Structure):
    _fields_ = [("op", C.c_int32), ("a", C.c_int32), ("b", C.c_int32), ("c", C.c_int32), ("imm", C.c_int64)]


class rdf_function(C.Structure):
    _fields_ = [("name", C.c_char_p), ("n_params", C.c_int32), ("n_exprs", C.c_int32),
                ("exprs", C.POINTER(rdf_expr)), ("root", C.c_int32), ("kind", C.c_int32), ("cond", C.c_int32),
                ("next", C.c_int32 * 3)]


class rdf_program(C.Structure):
    _fields_ = [("n_functions", C.c_int32), ("functions", C.POINTER(rdf_function)), ("result", C.c_int32),
                ("tag_mode", C.c_int32)]


class rdf_node(C.Structure):
    _fields_ = [("kind", C.c_int32), ("op", C.c_int32), ("label", C.c_int32), ("func", C.c_int32),
                ("param", C.c_int32), ("n_in", C.c_int32), ("value", C.c_int64)]


class rdf_edge(C.Structure):
    _fields_ = [("src", C.c_int32), ("src_port", C.c_int32), ("dst", C.c_int32), ("dst_port", C.c_int32),
                ("control", C.c_int32)]


class rdf_graph_desc(C.Structure):
    _fields_ = [("n_nodes", C.c_int32), ("n_edges", C.c_int32), ("nodes", C.POINTER(rdf_node)),
                ("edges", C.POINTER(rdf_edge)), ("n_labels", C.c_int32), ("label_bits", C.c_int32),
                ("n_match", C.c_int32), ("n_code", C.c_int32), ("label_callee", C.POINTER(C.c_int32)),
                ("label_local", C.POINTER(C.c_int32))]


class rdf_batch(C.Structure):
    _fields_ = [("B", C.c_int64), ("x", C.c_void_p), ("tree_root", C.c_void_p), ("N", C.c_int64),
                ("left", C.c_void_p), ("right", C.c_void_p), ("tok", C.c_void_p), ("label", C.c_void_p),
                ("max_invocations", C.c_int64), ("max_wave_tokens", C.c_int64)]


class rdf_params(C.Structure):
    _fields_ = [("compute", C.c_int32), ("H", C.c_int32), ("D", C.c_int32), ("V", C.c_int32),
                ("n_classes", C.c_int32), ("reproducible", C.c_int32), ("E", C.c_void_p), ("W", C.c_void_p), ("b", C.c_void_p),
                ("W_x", C.c_void_p), ("b_x", C.c_void_p), ("W_s", C.c_void_p), ("b_s", C.c_void_p)]


class rdf_trace_rec(C.Structure):
    _fields_ = [("tag", C.c_uint64), ("value", C.c_int64), ("kind", C.c_uint32), ("label", C.c_uint32),
                ("parent", C.c_uint32), ("instance", C.c_uint32)]


TRACE_DTYPE = np.dtype([("tag", "<u8"), ("value", "<i8"), ("kind", "<u4"), ("label", "<u4"), ("parent", "<u4"),
                        ("instance", "<u4")])


class rdf_outputs(C.Structure):
    _fields_ = [("y", C.c_void_p), ("h_root", C.c_void_p), ("loss", C.c_void_p), ("trace", C.c_void_p),
                ("trace_capacity", C.c_int64), ("trace_count", C.c_void_p)]


class rdf_param_grads(C.Structure):
    _fields_ = [("dE", C.c_void_p), ("dW", C.c_void_p), ("db", C.c_void_p), ("dW_x", C.c_void_p),
                ("db_x", C.c_void_p), ("dW_s", C.c_void_p), ("db_s", C.c_void_p)]


class rdf_stats(C.Structure):
    _fields_ = [("status", C.c_int32), ("waves", C.c_uint32), ("waves_backward", C.c_uint32),
                ("max_wave_tokens", C.c_uint32), ("invocations", C.c_uint64), ("tokens", C.c_uint64),
                ("store_inserts", C.c_uint64), ("store_matches", C.c_uint64), ("store_probes", C.c_uint64),
                ("max_probe", C.c_uint32), ("max_depth", C.c_uint32), ("cells", C.c_uint64), ("leaves", C.c_uint64),
                ("cycles_schedule", C.c_uint64), ("cycles_batch", C.c_uint64), ("cycles_barrier", C.c_uint64),
                ("cycles_bwd_frames", C.c_uint64), ("cycles_bwd_batch", C.c_uint64), ("cycles_bwd_barrier", C.c_uint64),
                ("kernel_launches", C.c_uint32), ("clusters", C.c_uint32)]

    def as_dict(self):
        return {k: getattr(self, k) for k, _ in self._fields_}


EXPORTS = ["rdf_graph_build", "rdf_graph_free", "rdf_graph_describe", "rdf_workspace_bytes", "rdf_eval", "rdf_grad",
           "rdf_last_status", "rdf_strerror", "rdf_set_profiling", "rdf_last_phase_ms", "rdf_eval_noalloc",
           "rdf_set_limits", "rdf_probe_fp32_fma", "rdf_set_store"]
PROBE_THREAD, PROBE_WARP = 0, 1
NOALLOC_SCRATCH_BYTES = 16 << 20
PHASES = ["setup", "schedule", "group", "operators", "roots", "loss", "lists", "backward", "dW", "db", "dE"]

_lib = None


def lib() -> C.CDLL:
    """Loads (building first if the sources are newer) the CUDA library."""
    global _lib
    if _lib is None:
        path = _build.build()
        L = C.CDLL(path)
        L.rdf_graph_build.argtypes = [C.POINTER(rdf_program), C.POINTER(C.c_void_p)]
        L.rdf_graph_free.argtypes = [C.c_void_p]
        L.rdf_graph_free.restype = None
        L.rdf_graph_describe.argtypes = [C.c_void_p, C.POINTER(rdf_graph_desc)]
        L.rdf_workspace_bytes.argtypes = [C.c_void_p, C.POINTER(rdf_batch), C.POINTER(rdf_params), C.c_int,
                                          C.POINTER(C.c_size_t)]
        L.rdf_eval.argtypes = [C.c_void_p, C.POINTER(rdf_batch), C.POINTER(rdf_params), C.POINTER(rdf_outputs),
                               C.c_void_p, C.c_size_t, C.c_void_p]
        L.rdf_grad.argtypes = [C.c_void_p, C.POINTER(rdf_batch), C.POINTER(rdf_params), C.POINTER(rdf_outputs),
                               C.POINTER(rdf_param_grads), C.c_void_p, C.c_size_t, C.c_void_p]
        L.rdf_eval_noalloc.argtypes = [C.c_void_p, C.POINTER(rdf_batch), C.POINTER(rdf_params),
                                       C.POINTER(rdf_outputs), C.c_void_p]
        L.rdf_last_status.argtypes = [C.c_void_p, C.POINTER(rdf_stats)]
        L.rdf_set_profiling.argtypes = [C.c_void_p, C.c_int]
        L.rdf_set_limits.argtypes = [C.c_void_p, C.c_longlong, C.c_longlong]
        L.rdf_set_store.argtypes = [C.c_void_p, C.c_int, C.c_longlong]
        L.rdf_probe_fp32_fma.argtypes = [C.POINTER(C.c_double), C.c_void_p]
        L.rdf_last_phase_ms.argtypes = [C.c_void_p, C.POINTER(C.c_float), C.c_int, C.POINTER(C.c_int)]
        L.rdf_strerror.argtypes = [C.c_int]
        L.rdf_strerror.restype = C.c_char_p
        _lib = L
    return _lib


def probe_fp32_fma_tflops() -> float:
    """fp32 FMA rate of the current CUDA device on a register-resident loop (TFLOP/s)."""
    torch = _torch()
    v = C.c_double()
    rc = lib().rdf_probe_fp32_fma(C.byref(v), torch.cuda.current_stream().cuda_stream)
    if rc != RDF_OK:
        raise RdfError(rc, "rdf_probe_fp32_fma")
    return float(v.value)


# ------------------------------------------------------- program description
class Function:
    """One definition as an expression list; methods return expression indices."""

    def __init__(self, name: str, n_params: int):
        self.name, self.n_params, self.exprs, self.root = name, n_params, [], -1
        self.kind, self.cond, self.next = FN_FUNCTION, -1, [-1, -1, -1]

    def loop(self, cond, nexts, value):
        """Makes this definition a while-loop over its parameters (the loop-carried variables): while `cond`, variable k
        becomes nexts[k]; at exit the loop's value is `value`.  A call of it with the initial values is the loop."""
        assert len(nexts) == self.n_params
        self.kind, self.cond, self.next, self.root = FN_LOOP, cond, list(nexts) + [-1] * (3 - len(nexts)), value
        return self

    def _add(self, op, a=-1, b=-1, c=-1, imm=0):
        self.exprs.append((op, a, b, c, imm))
        return len(self.exprs) - 1

    def param(self, k=0): return self._add(OP_PARAM, imm=k)
    def const(self, v): return self._add(OP_CONST, imm=int(v))
    def add(self, a, b): return self._add(OP_ADD, a, b)
    def sub(self, a, b): return self._add(OP_SUB, a, b)
    def mul(self, a, b): return self._add(OP_MUL, a, b)
    def max(self, a, b): return self._add(OP_MAX, a, b)
    def rem(self, a, b): return self._add(OP_REM, a, b)
    def lt(self, a, b): return self._add(OP_LT, a, b)
    def eq(self, a, b): return self._add(OP_EQ, a, b)
    def if_(self, c, a, b): return self._add(OP_IF, c, a, b)
    def call(self, f_index, *args): return self._add(OP_CALL, *(list(args) + [-1] * (3 - len(args))), imm=f_index)
    def is_leaf(self, v): return self._add(OP_IS_LEAF, v)
    def left(self, v): return self._add(OP_LEFT, v)
    def right(self, v): return self._add(OP_RIGHT, v)
    def tok(self, v): return self._add(OP_TOK, v)
    def embed(self, t): return self._add(OP_EMBED, t)
    def cell_rnn(self, a, b): return self._add(OP_CELL_RNN, a, b)
    def leaf_lstm(self, t): return self._add(OP_LEAF_LSTM, t)
    def cell_lstm(self, a, b): return self._add(OP_CELL_LSTM, a, b)
    def node_loss(self, s, v): return self._add(OP_NODE_LOSS, s, v)
    def child_l(self, h): return self._add(OP_CHILD_L, h)
    def child_r(self, h): return self._add(OP_CHILD_R, h)
    def gate(self, h): return self._add(OP_GATE, h)

    def ret(self, e):
        self.root = e
        return self


def fact_program(arg=3, addend=5):
    """result = addend + fact(arg); fact(n) = if 1 == n then n else n * fact(n-1)."""
    r = Function("result", 0)
    r.ret(r.add(r.const(addend), r.call(1, r.const(arg))))
    f = Function("fact", 1)
    n = f.param()
    f.ret(f.if_(f.eq(f.const(1), n), n, f.mul(n, f.call(1, f.sub(n, f.const(1))))))
    return [r, f], 0


def fib_program():
    """result(x) = fib(x); fib(n) = if n < 2 then n else fib(n-1) + fib(n-2)."""
    r = Function("result", 1)
    r.ret(r.call(1, r.param()))
    f = Function("fib", 1)
    n = f.param()
    f.ret(f.if_(f.lt(n, f.const(2)), n, f.add(f.call(1, f.sub(n, f.const(1))), f.call(1, f.sub(n, f.const(2))))))
    return [r, f], 0


def ack_program(m_const=2):
    """result(x) = ack(m_const, x); ack(m, n) = n+1 if m == 0, ack(m-1, 1) if n == 0, else ack(m-1, ack(m, n-1))."""
    r = Function("result", 1)
    r.ret(r.call(1, r.const(m_const), r.param()))
    f = Function("ack", 2)
    m, n = f.param(0), f.param(1)
    zero, one = f.const(0), f.const(1)
    m1 = f.sub(m, one)
    inner = f.call(1, m, f.sub(n, one))
    f.ret(f.if_(f.eq(m, zero), f.add(n, one), f.if_(f.eq(n, zero), f.call(1, m1, one), f.call(1, m1, inner))))
    return [r, f], 0


def primes_program():
    """result(x) = count(2, x), the number of primes <= x by trial division;
    count(i, n) = 0 if n < i else isprime(i, 2) + count(i + 1, n);
    isprime(i, d) = 1 if i < d * d, 0 if i % d == 0, else isprime(i, d + 1)."""
    r = Function("result", 1)
    r.ret(r.call(1, r.const(2), r.param()))
    c = Function("count", 2)
    i, n = c.param(0), c.param(1)
    c.ret(c.if_(c.lt(n, i), c.const(0), c.add(c.call(2, i, c.const(2)), c.call(1, c.add(i, c.const(1)), n))))
    q = Function("isprime", 2)
    i, d = q.param(0), q.param(1)
    q.ret(q.if_(q.lt(i, q.mul(d, d)), q.const(1),
                q.if_(q.eq(q.rem(i, d), q.const(0)), q.const(0), q.call(2, i, q.add(d, q.const(1))))))
    return [r, c, q], 0


def tak_program(y_const=12, z_const=6):
    """result(x) = tak(x, y, z); tak(x, y, z) = tak(tak(x-1, y, z), tak(y-1, z, x), tak(z-1, x, y)) if y < x else z."""
    r = Function("result", 1)
    r.ret(r.call(1, r.param(), r.const(y_const), r.const(z_const)))
    f = Function("tak", 3)
    x, y, z = f.param(0), f.param(1), f.param(2)
    one = f.const(1)
    a = f.call(1, f.sub(x, one), y, z)
    b = f.call(1, f.sub(y, one), z, x)
    c = f.call(1, f.sub(z, one), x, y)
    f.ret(f.if_(f.lt(y, x), f.call(1, a, b, c), z))
    return [r, f], 0


def topdown_program(depth_limit):
    """Recursion shaped by the values it computes (Section 6.2, last paragraph):
    result(v) = expand(seed(v), 0); seed(v) = EMBED(TOK(v));
    expand(h, d) = h if d >= D or GATE(h) else CELL_RNN(expand(left(h), d+1), expand(right(h), d+1));
    left(h) = CHILD_L(h); right(h) = CHILD_R(h)."""
    RESULT, SEED, EXPAND, LEFT, RIGHT = range(5)
    r = Function("result", 1)
    r.ret(r.call(EXPAND, r.call(SEED, r.param()), r.const(0)))
    s = Function("seed", 1)
    s.ret(s.embed(s.tok(s.param())))
    f = Function("expand", 2)
    h, d = f.param(0), f.param(1)
    d1 = f.add(d, f.const(1))
    stop = f.max(f.lt(f.const(depth_limit - 1), d), f.gate(h))
    f.ret(f.if_(stop, h, f.cell_rnn(f.call(EXPAND, f.call(LEFT, h), d1), f.call(EXPAND, f.call(RIGHT, h), d1))))
    fl = Function("left", 1)
    fl.ret(fl.child_l(fl.param()))
    fr = Function("right", 1)
    fr.ret(fr.child_r(fr.param()))
    return [r, s, f, fl, fr], RESULT


def find_program(threshold=50):
    """result(k) = find(k); find(k) = k if threshold < fib(k) else find(k + 1): the condition waits for a call."""
    RESULT, FIND, FIB = range(3)
    r = Function("result", 1)
    r.ret(r.call(FIND, r.param()))
    f = Function("find", 1)
    k = f.param()
    f.ret(f.if_(f.lt(f.const(threshold), f.call(FIB, k)), k, f.call(FIND, f.add(k, f.const(1)))))
    b = Function("fib", 1)
    n = b.param()
    b.ret(b.if_(b.lt(n, b.const(2)), n, b.add(b.call(FIB, b.sub(n, b.const(1))), b.call(FIB, b.sub(n, b.const(2))))))
    return [r, f, b], RESULT


def sum_loop_program():
    """result(n) = { s = 0; i = 0; while (i < n) { s = s + i; i = i + 1 }; s }: the while-loop of Figure 1."""
    r = Function("result", 1)
    r.ret(r.call(1, r.const(0), r.const(0), r.param()))
    lp = Function("sum_while", 3)
    s_, i, n = lp.param(0), lp.param(1), lp.param(2)
    lp.loop(lp.lt(i, n), [lp.add(s_, i), lp.add(i, lp.const(1)), n], s_)
    return [r, lp], 0


def pairs_loop_program():
    """result(n) = number of pairs (j, i), 0 <= j < i < n, by two nested loops (tags [j, i] in the inner one)."""
    r = Function("result", 1)
    r.ret(r.call(1, r.const(0), r.const(0), r.param()))
    outer = Function("outer", 3)
    acc, i, n = outer.param(0), outer.param(1), outer.param(2)
    outer.loop(outer.lt(i, n), [outer.call(2, acc, outer.const(0), i), outer.add(i, outer.const(1)), n], acc)
    inner = Function("inner", 3)
    a, j, lim = inner.param(0), inner.param(1), inner.param(2)
    inner.loop(inner.lt(j, lim), [inner.add(a, inner.const(1)), inner.add(j, inner.const(1)), lim], a)
    return [r, outer, inner], 0


def primes_loop_program():
    """result(x) = { c = 0; i = 2; while (not x < i) { c = c + isprime(i, 2); i = i + 1 }; c }: a recursive function
    called from a loop body."""
    r = Function("result", 1)
    r.ret(r.call(1, r.const(0), r.const(2), r.param()))
    lp = Function("count_while", 3)
    c, i, x = lp.param(0), lp.param(1), lp.param(2)
    lp.loop(lp.eq(lp.lt(x, i), lp.const(0)), [lp.add(c, lp.call(2, i, lp.const(2))), lp.add(i, lp.const(1)), x], c)
    q = Function("isprime", 2)
    i, d = q.param(0), q.param(1)
    q.ret(q.if_(q.lt(i, q.mul(d, d)), q.const(1),
                q.if_(q.eq(q.rem(i, d), q.const(0)), q.const(0), q.call(2, i, q.add(d, q.const(1))))))
    return [r, lp, q], 0


def tri_program():
    """result(x) = tri(x); tri(n) = 0 if n < 1 else sumto(n) + tri(n - 1), sumto a while-loop inside the recursive body."""
    r = Function("result", 1)
    r.ret(r.call(1, r.param()))
    f = Function("tri", 1)
    n = f.param()
    loop = f.call(2, f.const(0), f.const(0), n)
    f.ret(f.if_(f.lt(n, f.const(1)), f.const(0), f.add(loop, f.call(1, f.sub(n, f.const(1))))))
    lp = Function("sum_while", 3)
    s_, i, m = lp.param(0), lp.param(1), lp.param(2)
    lp.loop(lp.lt(i, m), [lp.add(s_, i), lp.add(i, lp.const(1)), m], s_)
    return [r, f, lp], 0


def tree_fold_program(kind: str):
    """Integer folds over the input trees: 'sum' of leaf tokens, leaf 'count', 'height'."""
    r = Function("result", 1)
    r.ret(r.call(1, r.param()))
    f = Function("fold", 1)
    v = f.param()
    a, b = f.call(1, f.left(v)), f.call(1, f.right(v))
    if kind == "sum":
        leaf, comb = f.tok(v), f.add(a, b)
    elif kind == "count":
        leaf, comb = f.const(1), f.add(a, b)
    else:
        leaf, comb = f.const(0), f.add(f.max(a, b), f.const(1))
    f.ret(f.if_(f.is_leaf(v), leaf, comb))
    return [r, f], 0


def tree_net_program(cell: str = "rnn", with_loss: bool = False):
    """h(v) = leaf(tok v) if is_leaf(v) else cell(h(left v), h(right v)), optionally under the per-node loss."""
    r = Function("result", 1)
    r.ret(r.call(1, r.param()))
    f = Function("h", 1)
    v = f.param()
    if cell == "rnn":
        body = f.if_(f.is_leaf(v), f.embed(f.tok(v)), f.cell_rnn(f.call(1, f.left(v)), f.call(1, f.right(v))))
    else:
        body = f.if_(f.is_leaf(v), f.leaf_lstm(f.tok(v)), f.cell_lstm(f.call(1, f.left(v)), f.call(1, f.right(v))))
    f.ret(f.node_loss(body, v) if with_loss else body)
    return [r, f], 0


# -------------------------------------------------------------------- graph
def _torch():
    import torch
    if not torch.cuda.is_available():
        raise RuntimeError("the recursive-dataflow library needs a CUDA device; there is no CPU path")
    return torch


class Graph:
    """A program transformed into one static graph and lowered for the device."""

    def __init__(self, functions, result=0, tag_mode=TAGS_PATH):
        self._keep = []
        fs = (rdf_function * len(functions))()
        for i, f in enumerate(functions):
            ex = (rdf_expr * max(1, len(f.exprs)))(*[rdf_expr(*e) for e in f.exprs])
            self._keep.append(ex)
            fs[i] = rdf_function(f.name.encode(), f.n_params, len(f.exprs), ex, f.root, f.kind, f.cond,
                                 (C.c_int32 * 3)(*f.next))
        prog = rdf_program(len(functions), fs, result, tag_mode)
        self.handle = C.c_void_p()
        self.tag_mode = tag_mode
        self._ws = None
        rc = lib().rdf_graph_build(C.byref(prog), C.byref(self.handle))
        if rc != RDF_OK:
            self.handle = None
            raise RdfError(rc, "rdf_graph_build")

    def __del__(self):
        if getattr(self, "handle", None):
            lib().rdf_graph_free(self.handle)
            self.handle = None

    def describe(self):
        d = rdf_graph_desc()
        rc = lib().rdf_graph_describe(self.handle, C.byref(d))
        if rc != RDF_OK:
            raise RdfError(rc, "rdf_graph_describe")
        nodes = [{k: getattr(d.nodes[i], k) for k, _ in rdf_node._fields_} for i in range(d.n_nodes)]
        edges = [{k: getattr(d.edges[i], k) for k, _ in rdf_edge._fields_} for i in range(d.n_edges)]
        return {"nodes": nodes, "edges": edges, "n_labels": d.n_labels, "label_bits": d.label_bits,
                "n_match": d.n_match, "n_code": d.n_code,
                "label_callee": [d.label_callee[i] for i in range(d.n_labels)],
                "label_local": [d.label_local[i] for i in range(d.n_labels)]}

    # ---- workspace (torch owns the memory)
    def workspace_bytes(self, batch, params, want_grad):
        n = C.c_size_t()
        rc = lib().rdf_workspace_bytes(self.handle, C.byref(batch), C.byref(params) if params else None, want_grad,
                                       C.byref(n))
        if rc != RDF_OK:
            raise RdfError(rc, "rdf_workspace_bytes")
        return n.value

    def _workspace(self, batch, params, want_grad):
        torch = _torch()
        n = self.workspace_bytes(batch, params, want_grad)
        if self._ws is None or self._ws.numel() < n + 256:
            self._ws = None
            self._ws = torch.empty(n + 256, dtype=torch.uint8, device="cuda")
        off = (-self._ws.data_ptr()) % 256
        return self._ws.data_ptr() + off, n

    def set_profiling(self, on=True):
        rc = lib().rdf_set_profiling(self.handle, int(on))
        if rc != RDF_OK:
            raise RdfError(rc, "rdf_set_profiling")

    def set_limits(self, wait_cycles=0, wave_limit=0):
        """Bound of the device-side waits (SM cycles) and of the number of scheduler waves; 0 = default."""
        rc = lib().rdf_set_limits(self.handle, int(wait_cycles), int(wave_limit))
        if rc != RDF_OK:
            raise RdfError(rc, "rdf_set_limits")

    def set_store(self, probe_mode=PROBE_THREAD, hash_slots=0):
        """Hash token store (path tags): probing strategy and slots per matching operator (0 = default)."""
        rc = lib().rdf_set_store(self.handle, int(probe_mode), int(hash_slots))
        if rc != RDF_OK:
            raise RdfError(rc, "rdf_set_store")

    def phase_ms(self):
        """{phase name: milliseconds} of the last call (needs set_profiling(True) before it)."""
        ms = (C.c_float * len(PHASES))()
        n = C.c_int()
        rc = lib().rdf_last_phase_ms(self.handle, ms, len(PHASES), C.byref(n))
        if rc != RDF_OK:
            raise RdfError(rc, "rdf_last_phase_ms")
        return {PHASES[k]: float(ms[k]) for k in range(n.value)}

    def stats(self, check=True):
        s = rdf_stats()
        rc = lib().rdf_last_status(self.handle, C.byref(s))
        if check and rc != RDF_OK:
            raise RdfError(rc, "device status")
        return s.as_dict()

    def _outputs(self, trace_capacity, **ptrs):
        torch = _torch()
        out = rdf_outputs()
        keep = None
        for k, v in ptrs.items():
            setattr(out, k, v.data_ptr() if v is not None else None)
        if trace_capacity:
            buf = torch.empty(trace_capacity * 32, dtype=torch.uint8, device="cuda")
            cnt = torch.zeros(1, dtype=torch.int64, device="cuda")
            out.trace, out.trace_capacity, out.trace_count = buf.data_ptr(), trace_capacity, cnt.data_ptr()
            keep = (buf, cnt)
        return out, keep

    @staticmethod
    def _read_trace(keep):
        if keep is None:
            return None
        buf, cnt = keep
        n = int(cnt.item())
        assert n * 32 <= buf.numel(), "trace buffer too small"
        return buf[: n * 32].cpu().numpy().view(TRACE_DTYPE)

    # ---- integer programs
    def eval_int(self, x, max_invocations, trace_capacity=0, max_wave_tokens=0, check=True, y=None):
        """x: int64 CUDA tensor [B].  Returns (y int64 CUDA tensor [B], trace ndarray or None)."""
        torch = _torch()
        assert x.is_cuda and x.dtype == torch.int64 and x.is_contiguous()
        B = x.numel()
        if y is None:
            y = torch.empty(B, dtype=torch.int64, device="cuda")
        batch = rdf_batch(B=B, x=x.data_ptr(), N=0, max_invocations=int(max_invocations),
                          max_wave_tokens=int(max_wave_tokens))
        out, tr = self._outputs(trace_capacity, y=y)
        ws, nbytes = self._workspace(batch, None, 0)
        rc = lib().rdf_eval(self.handle, C.byref(batch), None, C.byref(out), ws, nbytes,
                            torch.cuda.current_stream().cuda_stream)
        if rc != RDF_OK:
            raise RdfError(rc, "rdf_eval")
        if check:
            self.stats()
        return y, self._read_trace(tr)

    def eval_int_noalloc(self, x, y, max_invocations, check=True):
        """rdf_eval_noalloc for an integer program: the caller passes input x and output y (int64
        CUDA tensors of equal length); scratch is the library's built-in 16 MiB array, so nothing
        is allocated here -- not even through torch.  Raises RdfError(-3) when the batch needs more."""
        torch = _torch()
        assert x.is_cuda and y.is_cuda and x.dtype == y.dtype == torch.int64 and x.numel() == y.numel()
        batch = rdf_batch(B=x.numel(), x=x.data_ptr(), N=0, max_invocations=int(max_invocations), max_wave_tokens=0)
        out = rdf_outputs()
        out.y = y.data_ptr()
        rc = lib().rdf_eval_noalloc(self.handle, C.byref(batch), None, C.byref(out),
                                    torch.cuda.current_stream().cuda_stream)
        if rc != RDF_OK:
            raise RdfError(rc, "rdf_eval_noalloc")
        if check:
            self.stats()
        return y

    def eval_trees_noalloc(self, dt, dp, h_root, compute=F32, check=True):
        """rdf_eval_noalloc for a tree network: inputs dt/dp and the output h_root ([B, H] float32 CUDA
        tensor) are the caller's; scratch is the library's built-in array."""
        torch = _torch()
        batch = self._batch(dt)
        params = self._params(dp, compute)
        out = rdf_outputs()
        out.h_root = h_root.data_ptr()
        rc = lib().rdf_eval_noalloc(self.handle, C.byref(batch), C.byref(params), C.byref(out),
                                    torch.cuda.current_stream().cuda_stream)
        if rc != RDF_OK:
            raise RdfError(rc, "rdf_eval_noalloc")
        if check:
            self.stats()
        return h_root

    # ---- tree programs
    @staticmethod
    def device_trees(tb):
        """Uploads a workloads.TreeBatch; returns the dict of int32 CUDA tensors."""
        torch = _torch()
        return {k: torch.from_numpy(np.ascontiguousarray(getattr(tb, k), dtype=np.int32)).cuda()
                for k in ("tree_root", "left", "right", "tok", "label")}

    @staticmethod
    def device_params(params):
        torch = _torch()
        return {k: torch.from_numpy(np.ascontiguousarray(v, dtype=np.float32)).cuda() for k, v in params.items()}

    @staticmethod
    def _batch(dt):
        return rdf_batch(B=dt["tree_root"].numel(), x=None, tree_root=dt["tree_root"].data_ptr(),
                         N=dt["left"].numel(), left=dt["left"].data_ptr(), right=dt["right"].data_ptr(),
                         tok=dt["tok"].data_ptr(), label=dt["label"].data_ptr(), max_invocations=dt["left"].numel(),
                         max_wave_tokens=0)

    @staticmethod
    def _params(dp, compute, reproducible=False):
        g = lambda k: dp[k].data_ptr() if k in dp else None  # noqa: E731
        H = dp["W"].shape[1] // 2
        return rdf_params(compute=compute, H=H, D=dp["E"].shape[1], V=dp["E"].shape[0], reproducible=int(reproducible),
                          n_classes=dp["W_s"].shape[0] if "W_s" in dp else 0, E=g("E"), W=g("W"), b=g("b"),
                          W_x=g("W_x"), b_x=g("b_x"), W_s=g("W_s"), b_s=g("b_s"))

    def eval_trees(self, dt, dp, compute=F32, trace_capacity=0, check=True, h_root=None, max_invocations=None):
        """Forward pass over a batch of trees.  dt/dp: device_trees()/device_params().
        For integer tree programs (no parameters) pass dp=None: returns (y, trace)."""
        torch = _torch()
        batch = self._batch(dt)
        if max_invocations is not None:
            batch.max_invocations = int(max_invocations)
        B = batch.B
        if dp is None:
            y = torch.empty(B, dtype=torch.int64, device="cuda")
            out, tr = self._outputs(trace_capacity, y=y)
            params = None
        else:
            params = self._params(dp, compute)
            y = h_root if h_root is not None else torch.empty(B, params.H, dtype=torch.float32, device="cuda")
            out, tr = self._outputs(trace_capacity, h_root=y)
        ws, nbytes = self._workspace(batch, params, 0)
        rc = lib().rdf_eval(self.handle, C.byref(batch), C.byref(params) if params else None, C.byref(out), ws,
                            nbytes, torch.cuda.current_stream().cuda_stream)
        if rc != RDF_OK:
            raise RdfError(rc, "rdf_eval")
        if check:
            self.stats()
        return y, self._read_trace(tr)

    def grad_trees(self, dt, dp, compute=F32, check=True, grads=None, loss=None, h_root=None, max_invocations=None,
                   reproducible=False):
        """Forward + reverse pass.  Returns (loss tensor [1], h_root, {name: gradient tensor}).
        reproducible (BF16 only): bit-identical results on every call with the same inputs."""
        torch = _torch()
        batch = self._batch(dt)
        if max_invocations is not None:
            batch.max_invocations = int(max_invocations)
        params = self._params(dp, compute, reproducible)
        if h_root is None:
            h_root = torch.empty(batch.B, params.H, dtype=torch.float32, device="cuda")
        if loss is None:
            loss = torch.zeros(1, dtype=torch.float32, device="cuda")
        if grads is None:
            grads = {k: torch.empty_like(v) for k, v in dp.items()}
        pg = rdf_param_grads(**{"d" + k: grads[k].data_ptr() for k in grads})
        out, _ = self._outputs(0, h_root=h_root, loss=loss)
        ws, nbytes = self._workspace(batch, params, 1)
        rc = lib().rdf_grad(self.handle, C.byref(batch), C.byref(params), C.byref(out), C.byref(pg), ws, nbytes,
                            torch.cuda.current_stream().cuda_stream)
        if rc != RDF_OK:
            raise RdfError(rc, "rdf_grad")
        if check:
            self.stats()
        return loss, h_root, grads


# --------------------------------------------------------------- tag decode
def unpack_path_tag(tag: int, label_bits: int):
    """(instance, labels innermost first) of a packed 64-bit path tag."""
    tag = int(tag)
    inst = tag >> INST_SHIFT
    depth = (tag >> DEPTH_SHIFT) & 63
    path = tag & ((1 << PATH_BITS) - 1)
    return inst, tuple((path >> (label_bits * k)) & ((1 << label_bits) - 1) for k in range(depth))
