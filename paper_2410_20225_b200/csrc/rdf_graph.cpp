// Host side of the library: program validation, the graph transformation of
// Section 3 (recursive definitions -> one static graph with Call_i / Return_i),
// and the lowering of that graph into segments for the device executor.
#include <algorithm>
#include <climits>
#include <cstring>
#include <functional>
#include <map>
#include <set>

#include "rdf_internal.h"

namespace {

struct Err {
    int code;
};

inline void require(bool ok, int code) {
    if (!ok) throw Err{code};
}

int arity_of(int op) {
    switch (op) {
        case RDF_OP_PARAM: case RDF_OP_CONST: return 0;
        case RDF_OP_ADD: case RDF_OP_SUB: case RDF_OP_MUL: case RDF_OP_MAX:
        case RDF_OP_LT: case RDF_OP_EQ: case RDF_OP_REM: case RDF_OP_CELL_RNN: case RDF_OP_CELL_LSTM:
        case RDF_OP_NODE_LOSS: return 2;
        case RDF_OP_IF: return 3;
        case RDF_OP_CALL: case RDF_OP_IS_LEAF: case RDF_OP_LEFT: case RDF_OP_RIGHT: case RDF_OP_TOK:
        case RDF_OP_EMBED: case RDF_OP_LEAF_LSTM: case RDF_OP_CHILD_L: case RDF_OP_CHILD_R: case RDF_OP_GATE: return 1;
        default: return -1;
    }
}

struct Prog {
    const rdf_program* p;
    const rdf_function& fn(int i) const { return p->functions[i]; }
    const rdf_expr& ex(int f, int e) const { return p->functions[f].exprs[e]; }
    bool is_loop(int f) const { return p->functions[f].kind == RDF_FN_LOOP; }
    // number of operand expressions: a call has one per formal parameter of its callee
    int n_ops(const rdf_expr& x) const {
        if (x.op == RDF_OP_CALL) return (x.imm >= 0 && x.imm < p->n_functions) ? p->functions[x.imm].n_params : 0;
        return arity_of(x.op);
    }
};

// ---------------------------------------------------------------- validation
void validate(const Prog& P) {
    const rdf_program* p = P.p;
    require(p->n_functions > 0 && p->functions, RDF_ERR_BAD_PROGRAM);
    require(p->result >= 0 && p->result < p->n_functions, RDF_ERR_BAD_PROGRAM);
    require(p->tag_mode == RDF_TAGS_PATH || p->tag_mode == RDF_TAGS_FRAME, RDF_ERR_BAD_ARG);
    require(p->functions[p->result].n_params <= 1, RDF_ERR_UNSUPPORTED);    // one input per instance
    for (int f = 0; f < p->n_functions; ++f) {
        const rdf_function& F = p->functions[f];
        require(F.exprs && F.n_exprs > 0 && F.n_params >= 0 && F.name, RDF_ERR_BAD_PROGRAM);
        require(F.root >= 0 && F.root < F.n_exprs, RDF_ERR_BAD_PROGRAM);
        require(F.kind == RDF_FN_FUNCTION || F.kind == RDF_FN_LOOP, RDF_ERR_BAD_PROGRAM);
        if (F.kind == RDF_FN_LOOP) {
            require(f != p->result && F.n_params >= 1 && F.n_params <= 3, RDF_ERR_BAD_PROGRAM);
            require(F.cond >= 0 && F.cond < F.n_exprs, RDF_ERR_BAD_PROGRAM);
            for (int k = 0; k < F.n_params; ++k) require(F.next[k] >= 0 && F.next[k] < F.n_exprs, RDF_ERR_BAD_PROGRAM);
            require(p->tag_mode == RDF_TAGS_FRAME, RDF_ERR_UNSUPPORTED);     // the counter lives beside a frame id
        }
        for (int e = 0; e < F.n_exprs; ++e) {
            const rdf_expr& x = F.exprs[e];
            require(arity_of(x.op) >= 0, RDF_ERR_BAD_PROGRAM);
            if (x.op == RDF_OP_CALL) {
                require(x.imm >= 0 && x.imm < p->n_functions, RDF_ERR_BAD_PROGRAM);   // unknown callee
                require(x.imm != p->result, RDF_ERR_BAD_PROGRAM);
                const int m = p->functions[x.imm].n_params;
                require(m >= 1, RDF_ERR_BAD_PROGRAM);
                require(m <= 3, RDF_ERR_UNSUPPORTED);     // an expression node carries at most three operands
                // several parameters live in the invocation's frame: frame-form tags only
                require(m == 1 || p->tag_mode == RDF_TAGS_FRAME, RDF_ERR_UNSUPPORTED);
            }
            const int ar = P.n_ops(x);
            int ops[3] = {x.a, x.b, x.c};
            for (int k = 0; k < ar; ++k) require(ops[k] >= 0 && ops[k] < F.n_exprs, RDF_ERR_BAD_PROGRAM);   // arity mismatch too
            if (x.op == RDF_OP_PARAM) require(x.imm >= 0 && x.imm < F.n_params, RDF_ERR_BAD_PROGRAM);
        }
        // no cycles among expressions
        std::vector<int> state(F.n_exprs, 0);
        std::function<void(int)> dfs = [&](int e) {
            require(state[e] != 1, RDF_ERR_BAD_PROGRAM);
            if (state[e] == 2) return;
            state[e] = 1;
            const rdf_expr& x = F.exprs[e];
            int ops[3] = {x.a, x.b, x.c};
            for (int k = 0; k < P.n_ops(x); ++k) dfs(ops[k]);
            state[e] = 2;
        };
        dfs(F.root);
        if (F.kind == RDF_FN_LOOP) {
            dfs(F.cond);
            for (int k = 0; k < F.n_params; ++k) dfs(F.next[k]);
        }
    }
    // a loop stands in the graph of its caller: loops that contain themselves have no finite graph
    std::vector<int> lstate(p->n_functions, 0);
    std::function<void(int)> lwalk = [&](int f) {
        require(lstate[f] != 1, RDF_ERR_BAD_PROGRAM);
        if (lstate[f] == 2) return;
        lstate[f] = 1;
        const rdf_function& F = p->functions[f];
        for (int e = 0; e < F.n_exprs; ++e)
            if (F.exprs[e].op == RDF_OP_CALL && p->functions[F.exprs[e].imm].kind == RDF_FN_LOOP) lwalk((int)F.exprs[e].imm);
        lstate[f] = 2;
    };
    for (int f = 0; f < p->n_functions; ++f)
        if (p->functions[f].kind == RDF_FN_LOOP) lwalk(f);
}

// --------------------------------------------------------------- value kinds
// An expression is integer-valued or vector-valued (a state of the tree networks).  What the device
// executor supports: integer operators, conditions, accessors and call arguments take integers; a cell
// takes the results of two calls (it reads the states that the two callee invocations left in their
// frames), so an invocation fires at most one vector operator and a cell invocation makes exactly two
// calls -- which is what the per-invocation state slot and the sizing of the cell lists rely on.
// Anything else is a valid program that this executor does not lower: RDF_ERR_UNSUPPORTED.
void check_kinds(const Prog& P) {
    const int nf = P.p->n_functions;
    std::vector<int> fvec(nf, 0);                  // function returns a vector (fixpoint from "integer")
    std::vector<int> pvec(nf * 3, 0);              // formal parameter k of f is vector-valued: some call passes a state
    std::function<int(int, int)> kind = [&](int f, int e) -> int {
        const rdf_expr& x = P.ex(f, e);
        switch (x.op) {
            case RDF_OP_EMBED: case RDF_OP_LEAF_LSTM: case RDF_OP_CELL_RNN: case RDF_OP_CELL_LSTM:
            case RDF_OP_NODE_LOSS: case RDF_OP_CHILD_L: case RDF_OP_CHILD_R: return 1;
            case RDF_OP_PARAM: return pvec[f * 3 + (int)x.imm];
            case RDF_OP_CALL: return fvec[x.imm];
            case RDF_OP_IF: return kind(f, x.b) | kind(f, x.c);
            default: return 0;
        }
    };
    for (bool changed = true; changed;) {
        changed = false;
        for (int f = 0; f < nf; ++f) {
            const int k = kind(f, P.fn(f).root);
            if (k != fvec[f]) { fvec[f] = k; changed = true; }
            for (int e = 0; e < P.fn(f).n_exprs; ++e) {
                const rdf_expr& x = P.ex(f, e);
                if (x.op != RDF_OP_CALL) continue;
                const int ops[3] = {x.a, x.b, x.c};
                for (int k2 = 0; k2 < P.n_ops(x); ++k2)
                    if (kind(f, ops[k2]) && !pvec[(int)x.imm * 3 + k2]) { pvec[(int)x.imm * 3 + k2] = 1; changed = true; }
            }
        }
    }
    require(!pvec[P.p->result * 3], RDF_ERR_UNSUPPORTED);
    for (int f = 0; f < nf; ++f) {
        const rdf_function& F = P.fn(f);
        // at most one vector operator along any path through the body: the invocation's frame holds one state
        std::function<int(int)> vcount = [&](int e) -> int {
            const rdf_expr& x = F.exprs[e];
            if (x.op == RDF_OP_IF) return vcount(x.a) + std::max(vcount(x.b), vcount(x.c));
            int n = 0;
            switch (x.op) {
                case RDF_OP_EMBED: case RDF_OP_LEAF_LSTM: case RDF_OP_CELL_RNN: case RDF_OP_CELL_LSTM:
                case RDF_OP_CHILD_L: case RDF_OP_CHILD_R: n = 1; break;
                default: break;
            }
            if (x.op == RDF_OP_CALL) return 0;             // the operators of an argument that is a call run in the callee's frame;
                                                           // other arguments are checked below (integers, or plain parameters)
            const int ops[3] = {x.a, x.b, x.c};
            for (int k = 0; k < P.n_ops(x); ++k) n += vcount(ops[k]);
            return n;
        };
        require(vcount(F.root) <= 1, RDF_ERR_UNSUPPORTED);
        std::vector<char> seen(F.n_exprs, 0);
        std::function<void(int)> walk = [&](int e) {
            if (seen[e]) return;
            seen[e] = 1;
            const rdf_expr& x = F.exprs[e];
            const int ops[3] = {x.a, x.b, x.c};
            const int n = P.n_ops(x);
            for (int k = 0; k < n; ++k) walk(ops[k]);
            switch (x.op) {
                case RDF_OP_IF:
                    require(kind(f, x.a) == 0, RDF_ERR_UNSUPPORTED);                 // a Switch takes an integer (RDF_OP_GATE makes one)
                    require(kind(f, x.b) == kind(f, x.c), RDF_ERR_UNSUPPORTED);
                    break;
                case RDF_OP_CELL_RNN: case RDF_OP_CELL_LSTM:
                    for (int k = 0; k < 2; ++k)                                          // operands: states of two callees
                        require(F.exprs[ops[k]].op == RDF_OP_CALL && kind(f, ops[k]) == 1, RDF_ERR_UNSUPPORTED);
                    break;
                case RDF_OP_NODE_LOSS:
                    require(kind(f, x.a) == 1 && kind(f, x.b) == 0, RDF_ERR_UNSUPPORTED);
                    break;
                case RDF_OP_CHILD_L: case RDF_OP_CHILD_R: case RDF_OP_GATE:
                    // reads a state that exists when the invocation starts: a vector-valued parameter
                    require(F.exprs[x.a].op == RDF_OP_PARAM && kind(f, x.a) == 1, RDF_ERR_UNSUPPORTED);
                    require(P.p->tag_mode == RDF_TAGS_FRAME, RDF_ERR_UNSUPPORTED);
                    break;
                case RDF_OP_CALL:
                    // an argument is of the kind the callee's parameter has at every call site; a state is passed on as a
                    // parameter or as the result of a call (by reference), never computed in the argument itself
                    for (int k = 0; k < n; ++k) {
                        require(kind(f, ops[k]) == pvec[(int)x.imm * 3 + k], RDF_ERR_UNSUPPORTED);
                        if (kind(f, ops[k]))
                            require(F.exprs[ops[k]].op == RDF_OP_PARAM || F.exprs[ops[k]].op == RDF_OP_CALL, RDF_ERR_UNSUPPORTED);
                    }
                    require(!(P.is_loop((int)x.imm) && (pvec[(int)x.imm * 3] | pvec[(int)x.imm * 3 + 1] | pvec[(int)x.imm * 3 + 2])),
                            RDF_ERR_UNSUPPORTED);
                    break;
                default:                                                                 // integer operands only
                    for (int k = 0; k < n; ++k) require(kind(f, ops[k]) == 0, RDF_ERR_UNSUPPORTED);
            }
        };
        walk(F.root);
        if (F.kind == RDF_FN_LOOP) {
            walk(F.cond);
            for (int k = 0; k < F.n_params; ++k) walk(F.next[k]);
            require(kind(f, F.root) == 0 && kind(f, F.cond) == 0, RDF_ERR_UNSUPPORTED);      // integer loops
            for (int k = 0; k < F.n_params; ++k) require(kind(f, F.next[k]) == 0, RDF_ERR_UNSUPPORTED);
            // the condition and the value at exit are evaluated where the variables are at hand: no calls in them
            std::function<bool(int)> has_call = [&](int e) {
                const rdf_expr& x = F.exprs[e];
                if (x.op == RDF_OP_CALL) return true;
                const int ops[3] = {x.a, x.b, x.c};
                for (int k = 0; k < P.n_ops(x); ++k)
                    if (has_call(ops[k])) return true;
                return false;
            };
            require(!has_call(F.cond) && !has_call(F.root), RDF_ERR_UNSUPPORTED);
        }
    }
}

// ------------------------------------------------- literal graph (Section 3)
const int NODE_FCALL = 100;   // placeholder: a function-call node of Section 2.4 (replaced by Call_i / Return_i)

struct Literal {
    const Prog& P;
    std::vector<rdf_node>& nodes;
    std::vector<rdf_edge>& edges;
    std::vector<int> in_node;    // per function: first IN node
    std::vector<int> out_node;   // per function: OUT node
    std::vector<int64_t> callee; // per node: callee of an FCALL placeholder

    int add(int kind, int op, int func, int n_in, int64_t value = 0, int param = 0) {
        rdf_node n;
        n.kind = kind; n.op = op; n.label = -1; n.func = func; n.param = param; n.n_in = n_in; n.value = value;
        nodes.push_back(n);
        callee.push_back(-1);
        return (int)nodes.size() - 1;
    }
    void connect(int src, int sp, int dst, int dp, int control = 0) {
        edges.push_back(rdf_edge{src, sp, dst, dp, control});
    }

    uint32_t params_used(int f, int e, std::map<int, uint32_t>& memo) {
        auto it = memo.find(e);
        if (it != memo.end()) return it->second;
        const rdf_expr& x = P.ex(f, e);
        uint32_t m = 0;
        if (x.op == RDF_OP_PARAM) m = 1u << x.imm;
        int ops[3] = {x.a, x.b, x.c};
        for (int k = 0; k < P.n_ops(x); ++k) m |= params_used(f, ops[k], memo);
        memo[e] = m;
        return m;
    }

    typedef std::pair<int, int> Val;   // (node, output port)
    struct Gate {
        Val pred;
        int side;          // Switch output that is live in this context
        bool conditional;  // the predicate reads a parameter, so it is itself live only in its own context
    };
    struct Ctx {
        int id;
        std::vector<Val> param;
        std::vector<Gate> gates;   // enclosing conditionals, outermost first
    };

    void build_function(int f) {
        const rdf_function& F = P.fn(f);
        Ctx root{0, {}, {}};
        in_node[f] = (int)nodes.size();
        for (int k = 0; k < F.n_params; ++k) root.param.push_back(Val(add(RDF_NODE_IN, -1, f, 0, 0, k), 0));
        std::map<std::pair<int, int>, Val> memo;             // (expression, context): a context belongs to one definition
        std::map<int, std::map<int, uint32_t>> used;         // per definition
        int next_ctx = 1;
        // fn: the definition whose expression e is built (f itself, or a loop that stands inside f's graph)
        std::function<Val(int, int, const Ctx&)> build = [&](int fn, int e, const Ctx& c) -> Val {
            auto key = std::make_pair(e, c.id);
            auto it = memo.find(key);
            if (it != memo.end()) return it->second;
            const rdf_function& G = P.fn(fn);
            const rdf_expr& x = G.exprs[e];
            Val v;
            if (x.op == RDF_OP_PARAM) {
                v = c.param[x.imm];
            } else if (x.op == RDF_OP_CONST) {
                v = Val(add(RDF_NODE_CONST, -1, f, 0, x.imm), 0);
            } else if (x.op == RDF_OP_IF) {
                // Figure 2: the predicate drives a Switch that routes the parameter to one side
                Val pred = build(fn, x.a, c);
                uint32_t m = params_used(fn, x.b, used[fn]) | params_used(fn, x.c, used[fn]);
                Ctx ct{next_ctx++, c.param, c.gates}, cf{next_ctx++, c.param, c.gates};
                const bool conditional = params_used(fn, x.a, used[fn]) != 0;
                ct.gates.push_back(Gate{pred, 0, conditional});
                cf.gates.push_back(Gate{pred, 1, conditional});
                for (int k = 0; k < G.n_params; ++k) {
                    if (!(m >> k & 1)) continue;
                    int sw = add(RDF_NODE_SWITCH, -1, f, 2);
                    connect(pred.first, pred.second, sw, 0);
                    connect(c.param[k].first, c.param[k].second, sw, 1);
                    ct.param[k] = Val(sw, 0);
                    cf.param[k] = Val(sw, 1);
                }
                Val a = build(fn, x.b, ct), b = build(fn, x.c, cf);
                // a side that reads no parameter (a bare constant) would fire under every
                // tag; route its value through a Switch so that only the chosen side is live
                if (params_used(fn, x.b, used[fn]) == 0) {
                    int sw = add(RDF_NODE_SWITCH, -1, f, 2);
                    connect(pred.first, pred.second, sw, 0);
                    connect(a.first, a.second, sw, 1);
                    a = Val(sw, 0);
                }
                if (params_used(fn, x.c, used[fn]) == 0) {
                    int sw = add(RDF_NODE_SWITCH, -1, f, 2);
                    connect(pred.first, pred.second, sw, 0);
                    connect(b.first, b.second, sw, 1);
                    b = Val(sw, 1);
                }
                int mg = add(RDF_NODE_MERGE, -1, f, 2);
                connect(a.first, a.second, mg, 0);
                connect(b.first, b.second, mg, 1);
                v = Val(mg, 0);
            } else if (x.op == RDF_OP_CALL) {
                const int m = P.n_ops(x);
                const int ops[3] = {x.a, x.b, x.c};
                Val in[3];
                for (int k = 0; k < m; ++k) {
                    in[k] = build(fn, ops[k], c);
                    // an argument that reads no parameter would feed its Call_i under every tag of
                    // this function: let the enclosing conditionals' Switches pass it on instead
                    if (params_used(fn, ops[k], used[fn]) != 0) continue;
                    for (int gi = (int)c.gates.size() - 1; gi >= 0; --gi) {
                        const Gate& gt = c.gates[gi];
                        int sw = add(RDF_NODE_SWITCH, -1, f, 2);
                        connect(gt.pred.first, gt.pred.second, sw, 0);
                        connect(in[k].first, in[k].second, sw, 1);
                        in[k] = Val(sw, gt.side);
                        if (gt.conditional) break;
                    }
                }
                if (P.is_loop((int)x.imm)) {
                    // The while-loop of Figure 1 in place of the call: per loop-carried variable an Enter, a Merge fed by
                    // Enter and Next, a Switch on the condition; the body on the true side ends in Next, the value on
                    // the false side leaves through Exit.
                    const int lp = (int)x.imm;
                    const rdf_function& Lf = P.fn(lp);
                    const int first_new = (int)nodes.size();
                    Ctx cm{next_ctx++, {}, {}};
                    std::vector<int> merges;
                    for (int k = 0; k < m; ++k) {
                        int en = add(RDF_NODE_ENTER, -1, f, 1, 0, k);
                        connect(in[k].first, in[k].second, en, 0);
                        int mg = add(RDF_NODE_MERGE, -1, f, 2, 0, k);
                        connect(en, 0, mg, 0);
                        merges.push_back(mg);
                        cm.param.push_back(Val(mg, 0));
                    }
                    Val pred = build(lp, Lf.cond, cm);
                    Ctx ct{next_ctx++, {}, {Gate{pred, 0, true}}}, cf{next_ctx++, {}, {Gate{pred, 1, true}}};
                    for (int k = 0; k < m; ++k) {
                        int sw = add(RDF_NODE_SWITCH, -1, f, 2);
                        connect(pred.first, pred.second, sw, 0);
                        connect(merges[k], 0, sw, 1);
                        ct.param.push_back(Val(sw, 0));
                        cf.param.push_back(Val(sw, 1));
                    }
                    for (int k = 0; k < m; ++k) {
                        Val nv = build(lp, Lf.next[k], ct);
                        int nx = add(RDF_NODE_NEXT, -1, f, 1, 0, k);
                        connect(nv.first, nv.second, nx, 0);
                        connect(nx, 0, merges[k], 1);
                    }
                    Val rv = build(lp, Lf.root, cf);
                    int ex = add(RDF_NODE_EXIT, -1, f, 1);
                    connect(rv.first, rv.second, ex, 0);
                    // a constant inside the loop emits once per iteration, under the iteration's tag: fired by the Merge
                    // (param = 1 marks it as fired by a loop, not by the entry Merge of the enclosing function)
                    for (int n = first_new; n < (int)nodes.size(); ++n)
                        if (nodes[n].kind == RDF_NODE_CONST && nodes[n].param == 0) {
                            nodes[n].param = 1;
                            connect(merges[0], 0, n, -1, 1);
                        }
                    v = Val(ex, 0);
                } else {
                    int n = add(NODE_FCALL, -1, f, m);
                    callee[n] = x.imm;
                    for (int k = 0; k < m; ++k) connect(in[k].first, in[k].second, n, k);
                    v = Val(n, 0);
                }
            } else {
                int ar = arity_of(x.op);
                int ops[3] = {x.a, x.b, x.c};
                Val in[3];
                for (int k = 0; k < ar; ++k) in[k] = build(fn, ops[k], c);
                int n = add(RDF_NODE_OP, x.op, f, ar);
                for (int k = 0; k < ar; ++k) connect(in[k].first, in[k].second, n, k);
                v = Val(n, 0);
            }
            memo[key] = v;
            return v;
        };
        Val r = build(f, F.root, root);
        out_node[f] = add(RDF_NODE_OUT, -1, f, 1);
        connect(r.first, r.second, out_node[f], 0);
    }

    // The five steps of the general algorithm, per callee f.
    void transform() {
        const int nf = P.p->n_functions;
        std::set<int> removed;
        for (int f = 0; f < nf; ++f) {
            if (f == P.p->result || P.is_loop(f)) continue;
            const int m = P.fn(f).n_params;
            // 1. number the nodes that call f: 0 .. n-1 (callers in `result` first)
            std::vector<int> calls;
            for (int n = 0; n < (int)nodes.size(); ++n)
                if (nodes[n].kind == NODE_FCALL && callee[n] == f) calls.push_back(n);
            std::stable_sort(calls.begin(), calls.end(), [&](int a, int b) {
                return (nodes[a].func == P.p->result) > (nodes[b].func == P.p->result);
            });
            const int n_calls = (int)calls.size();
            if (n_calls == 0) continue;
            // 3. input nodes become Merge nodes with one input per call site
            for (int k = 0; k < m; ++k) {
                rdf_node& in = nodes[in_node[f] + k];
                in.kind = RDF_NODE_ENTRY_MERGE;
                in.n_in = n_calls;
            }
            // the edge into f's output node
            rdf_edge out_edge{};
            for (const rdf_edge& e : edges)
                if (e.dst == out_node[f]) out_edge = e;
            removed.insert(out_node[f]);
            for (int i = 0; i < n_calls; ++i) {
                const int c = calls[i];
                // 2. m Call_i nodes, one per formal parameter, each with its one input
                std::vector<int> call_nodes;
                for (int k = 0; k < m; ++k) {
                    rdf_edge arg{};
                    for (const rdf_edge& e : edges)
                        if (e.dst == c && e.dst_port == k) arg = e;
                    int cn = add(RDF_NODE_CALL, -1, nodes[c].func, 1, 0, k);
                    nodes[cn].label = i;
                    callee[cn] = f;
                    connect(arg.src, arg.src_port, cn, 0);
                    connect(cn, 0, in_node[f] + k, i);
                    call_nodes.push_back(cn);
                }
                // 4. Return_i after f's output, feeding the consumers of call node i
                int rn = add(RDF_NODE_RETURN, -1, nodes[c].func, 1);
                nodes[rn].label = i;
                callee[rn] = f;
                connect(out_edge.src, out_edge.src_port, rn, 0);
                const size_t n_edges = edges.size();
                for (size_t j = 0; j < n_edges; ++j)
                    if (edges[j].src == c) connect(rn, 0, edges[j].dst, edges[j].dst_port, edges[j].control);
                // 5. control edge Call_i -> Return_i
                for (int cn : call_nodes) connect(cn, 0, rn, -1, 1);
                removed.insert(c);
            }
            // Figure 3: constants of a called function fire on its entry Merge
            for (int n = 0; n < (int)nodes.size(); ++n)
                if (nodes[n].kind == RDF_NODE_CONST && nodes[n].func == f && nodes[n].param == 0) connect(in_node[f], 0, n, -1, 1);
        }
        // drop replaced nodes, renumber
        std::vector<int> new_id(nodes.size(), -1);
        std::vector<rdf_node> keep;
        for (int n = 0; n < (int)nodes.size(); ++n)
            if (!removed.count(n)) {
                new_id[n] = (int)keep.size();
                keep.push_back(nodes[n]);
            }
        std::vector<rdf_edge> kept;
        for (const rdf_edge& e : edges)
            if (new_id[e.src] >= 0 && new_id[e.dst] >= 0)
                kept.push_back(rdf_edge{new_id[e.src], e.src_port, new_id[e.dst], e.dst_port, e.control});
        nodes.swap(keep);
        edges.swap(kept);
    }
};

void build_literal(const Prog& P, rdf_graph* g) {
    Literal L{P, g->nodes, g->edges, {}, {}, {}};
    const int nf = P.p->n_functions;
    L.in_node.assign(nf, -1);
    L.out_node.assign(nf, -1);
    L.build_function(P.p->result);          // `result` first, as the paper draws it
    for (int f = 0; f < nf; ++f)
        if (f != P.p->result && !P.is_loop(f)) L.build_function(f);      // (a loop stands inside the graphs that use it)
    L.transform();
}

// ------------------------------------------------------------------ lowering
struct Seg {
    std::vector<VmInstr> code;
    int nregs = 0;
    std::map<int, int> memo;     // expression -> register (only valid in an entry segment)
    bool entry = false;
    int base = -1;               // absolute pc after layout
};

struct Cont {
    int kind;                    // 0 RET, 1 OUT, 2 PORT, 3 CODE
    int node = 0, port = 0;
    std::function<void(int seg, int reg)> fn;
};

struct Lower {
    const Prog& P;
    rdf_graph* g;
    std::vector<Seg> segs;
    std::vector<int> entry_seg;          // per function
    std::vector<int> label_entry_seg;    // per label: callee's entry segment
    std::vector<int> label_kseg;         // per label: continuation segment (K_SEG) or -1
    std::vector<int> match_cont_seg;     // per match node
    std::vector<int> local_count;        // per callee: call sites numbered so far
    int cur_func = 0;
    int calls_in_body = 0;

    int new_seg() {
        segs.emplace_back();
        return (int)segs.size() - 1;
    }
    int reg(int s) {
        require(segs[s].nregs < RDF_MAX_REGS, RDF_ERR_UNSUPPORTED);
        return segs[s].nregs++;
    }
    void emit(int s, uint8_t op, int dst = 0, int a = 0, int b = 0, int32_t imm = 0) {
        segs[s].code.push_back(VmInstr{op, (uint8_t)dst, (uint8_t)a, (uint8_t)b, imm});
    }

    bool call_free(int f, int e) {
        const rdf_expr& x = P.ex(f, e);
        switch (x.op) {
            case RDF_OP_CALL: case RDF_OP_EMBED: case RDF_OP_LEAF_LSTM: case RDF_OP_CELL_RNN:
            case RDF_OP_CELL_LSTM: case RDF_OP_NODE_LOSS: case RDF_OP_CHILD_L: case RDF_OP_CHILD_R: return false;
            default: break;
        }
        int ops[3] = {x.a, x.b, x.c};
        for (int k = 0; k < P.n_ops(x); ++k)
            if (!call_free(f, ops[k])) return false;
        return true;
    }

    int load_const(int s, int64_t v) {
        int r = reg(s);
        if (v >= INT32_MIN && v <= INT32_MAX) {
            emit(s, VM_MOVI, r, 0, 0, (int32_t)v);
        } else {
            require((int)g->consts.size() < RDF_MAX_CONSTS, RDF_ERR_UNSUPPORTED);
            g->consts.push_back(v);
            emit(s, VM_MOVC, r, 0, 0, (int32_t)g->consts.size() - 1);
        }
        return r;
    }

    uint8_t vm_binop(int op) {
        switch (op) {
            case RDF_OP_ADD: return VM_ADD; case RDF_OP_SUB: return VM_SUB; case RDF_OP_MUL: return VM_MUL;
            case RDF_OP_MAX: return VM_MAX; case RDF_OP_LT: return VM_LT; case RDF_OP_EQ: return VM_EQ;
            case RDF_OP_REM: return VM_REM;
        }
        throw Err{RDF_ERR_UNSUPPORTED};
    }

    // value of a call-free expression, computed where the parameters are live
    int value(int s, int e) {
        auto it = segs[s].memo.find(e);
        if (it != segs[s].memo.end()) return it->second;
        const rdf_expr& x = P.ex(cur_func, e);
        int r;
        switch (x.op) {
            case RDF_OP_PARAM:
                if (segs[s].entry) {                           // parameters are in registers in an entry segment
                    r = (int)x.imm;
                } else {
                    // elsewhere (the code after a condition that waited for a call) they are read back from the invocation's
                    // frame: frame-form tags, and not inside a loop (whose variables change from iteration to iteration)
                    require(P.p->tag_mode == RDF_TAGS_FRAME && !P.is_loop(cur_func), RDF_ERR_UNSUPPORTED);
                    r = reg(s);
                    emit(s, VM_LDARG, r, 0, 0, (int32_t)x.imm);
                    if (x.imm > 0) g->max_params = std::max(g->max_params, 2);
                }
                break;
            case RDF_OP_CONST: r = load_const(s, x.imm); break;
            case RDF_OP_IS_LEAF: case RDF_OP_LEFT: case RDF_OP_RIGHT: case RDF_OP_TOK: {
                int a = value(s, x.a);
                r = reg(s);
                g->uses_tree = true;
                emit(s, x.op == RDF_OP_IS_LEAF ? VM_ISLEAF : x.op == RDF_OP_LEFT ? VM_LEFT
                        : x.op == RDF_OP_RIGHT ? VM_RIGHT : VM_TOK, r, a);
                break;
            }
            case RDF_OP_GATE: {
                int a = value(s, x.a);
                r = reg(s);
                g->interleaved = true;
                emit(s, VM_VGATE, r, a);
                break;
            }
            case RDF_OP_IF: {
                // both sides call-free: an ordinary branch that joins
                int c = value(s, x.a);
                r = reg(s);
                std::map<int, int> saved = segs[s].memo;   // values computed in one arm are not live in the other
                size_t brz = segs[s].code.size();
                emit(s, VM_BRZ, 0, c);
                int a = value(s, x.b);
                emit(s, VM_MOV, r, a);
                size_t jmp = segs[s].code.size();
                emit(s, VM_JMP);
                segs[s].memo = saved;
                segs[s].code[brz].imm = (int32_t)segs[s].code.size();
                int b = value(s, x.c);
                emit(s, VM_MOV, r, b);
                segs[s].code[jmp].imm = (int32_t)segs[s].code.size();
                segs[s].memo = saved;
                break;
            }
            default: {
                int a = value(s, x.a), b = value(s, x.b);
                r = reg(s);
                emit(s, vm_binop(x.op), r, a, b);
            }
        }
        segs[s].memo[e] = r;
        return r;
    }

    void apply(const Cont& K, int s, int r) {
        switch (K.kind) {
            case 0: emit(s, VM_RET, 0, r); break;
            case 1: emit(s, VM_OUT, 0, r); break;
            case 2: emit(s, VM_PORT, 0, r, K.port, K.node); break;
            default: K.fn(s, r);
        }
    }

    // a fresh segment that receives one value in r0 and hands it to K
    int cont_segment(const Cont& K) {
        int s = new_seg();
        int r0 = reg(s);
        apply(K, s, r0);
        emit(s, VM_HALT);
        return s;
    }

    int new_label(int callee, const Cont& K) {
        require((int)g->labels.size() < RDF_MAX_LABELS, RDF_ERR_UNSUPPORTED);
        LabelInfo L{};
        L.callee = callee;
        L.local_label = local_count[callee]++;
        L.child_index = calls_in_body++;
        L.n_args = P.fn(callee).n_params;
        int kseg = -1;
        if (K.kind == 2) {
            L.k_kind = K_PORT; L.k_node = K.node; L.k_port = K.port;
        } else if (K.kind == 0) {
            L.k_kind = K_RET;
        } else {
            L.k_kind = K_SEG;
            kseg = cont_segment(K);
        }
        g->labels.push_back(L);
        label_entry_seg.push_back(entry_seg[callee]);
        label_kseg.push_back(kseg);
        return (int)g->labels.size() - 1;
    }

    int new_match(int n_ports, int kind, int cont_seg) {
        require((int)g->match.size() < RDF_MAX_MATCH, RDF_ERR_UNSUPPORTED);
        MatchNode M{n_ports, kind, 0, g->n_ports_total};
        g->n_ports_total += n_ports;
        g->match.push_back(M);
        match_cont_seg.push_back(cont_seg);
        return (int)g->match.size() - 1;
    }

    // The while-loop `lp` at this place of segment s, entered with the variables in registers r[0 .. m): Enter makes the
    // loop frame and sends the first iteration to the loop head (a segment of its own, run once per iteration, with the
    // variables in r0 .. r(m-1) like the parameters of a function entry).  There: the condition; while it holds, the next
    // values (from this segment, or gathered in the token store when some of them wait for calls) and Next; when it
    // fails, the value, Exit and what the enclosing code does with it (K).
    void emit_loop(int s, int lp, const int r[3], const Cont& K) {
        const rdf_function& Lf = P.fn(lp);
        const int m = Lf.n_params;
        g->has_loops = true;
        const int head = new_seg();
        segs[head].entry = true;
        segs[head].nregs = std::max(1, m);
        emit(s, VM_ENTER, r[2], r[0], r[1], -(head + 1));                  // (target fixed up at layout)
        const int outer = cur_func;
        cur_func = lp;
        for (int k = 1; k < m; ++k) emit(head, VM_LDARG, k, 0, 0, k);        // variables 1, 2 live in the loop frame
        const int c = value(head, Lf.cond);
        const std::map<int, int> saved = segs[head].memo;                   // values of the body are not live after the exit
        const size_t brz = segs[head].code.size();
        emit(head, VM_BRZ, 0, c);
        bool all_free = true;
        for (int k = 0; k < m; ++k) all_free = all_free && call_free(lp, Lf.next[k]);
        if (all_free) {
            int nr[3] = {0, 0, 0};
            for (int k = 0; k < m; ++k) nr[k] = value(head, Lf.next[k]);
            emit(head, VM_NEXT, nr[2], nr[0], nr[1], -(head + 1));
        } else if (m == 1) {
            // the one next value waits for a call: Next fires where that value arrives
            Cont K1{3};
            K1.fn = [this, head](int s2, int rv) { emit(s2, VM_NEXT, 0, rv, 0, -(head + 1)); };
            cps(head, Lf.next[0], K1);
            emit(head, VM_HALT);
        } else {
            // some next value waits for a call: the m values meet in the token store under the iteration's tag
            const int ks = new_seg();
            int rr[3] = {0, 0, 0};
            for (int k = 0; k < m; ++k) rr[k] = reg(ks);
            emit(ks, VM_NEXT, rr[2], rr[0], rr[1], -(head + 1));
            emit(ks, VM_HALT);
            const int M = new_match(m, MATCH_INT, ks);
            for (int k = 0; k < m; ++k) {
                Cont Kk{2, M, k};
                cps(head, Lf.next[k], Kk);
            }
            emit(head, VM_HALT);
        }
        segs[head].memo = saved;
        segs[head].code[brz].imm = (int32_t)segs[head].code.size();
        const int rv = value(head, Lf.root);
        emit(head, VM_EXIT);
        cur_func = outer;
        apply(K, head, rv);
        emit(head, VM_HALT);
    }

    // start the evaluation of expression e in segment s; its value goes to K
    void cps(int s, int e, const Cont& K) {
        const int f = cur_func;
        if (call_free(f, e)) {
            apply(K, s, value(s, e));
            return;
        }
        const rdf_expr& x = P.ex(f, e);
        switch (x.op) {
            case RDF_OP_CALL: {
                const int callee = (int)x.imm;
                const int m = P.n_ops(x);
                const int ops[3] = {x.a, x.b, x.c};
                bool all_free = true;
                for (int k = 0; k < m; ++k) all_free = all_free && call_free(f, ops[k]);
                const bool loop = P.is_loop(callee);
                if (all_free) {
                    // the m Call_i nodes of this call site fire together: all arguments are at hand
                    int r[3] = {0, 0, 0};
                    for (int k = 0; k < m; ++k) r[k] = value(s, ops[k]);
                    if (loop) {
                        emit_loop(s, callee, r, K);
                        break;
                    }
                    int label = new_label(callee, K);
                    emit(s, VM_CALL, r[2], r[0], r[1], label);
                } else if (m == 1) {
                    Cont K2{3};
                    K2.fn = [this, callee, K, loop](int s2, int r) {
                        if (loop) {
                            const int rr[3] = {r, 0, 0};
                            emit_loop(s2, callee, rr, K);
                            return;
                        }
                        int label = new_label(callee, K);
                        emit(s2, VM_CALL, 0, r, 0, label);
                    };
                    cps(s, x.a, K2);
                } else if (loop) {
                    // initial values that wait for calls meet in the token store; the loop is entered when the last has arrived
                    int ks = new_seg();
                    int r[3] = {0, 0, 0};
                    for (int k = 0; k < m; ++k) r[k] = reg(ks);
                    int M = new_match(m, MATCH_INT, ks);
                    for (int k = 0; k < m; ++k) {
                        Cont Kk{2, M, k};
                        cps(s, ops[k], Kk);
                    }
                    emit_loop(ks, callee, r, K);
                    emit(ks, VM_HALT);
                } else {
                    // some argument is itself the result of a call: the arguments meet in the token store
                    // under the caller's tag, and the call fires when the last one has arrived
                    int ks = new_seg();
                    int r[3] = {0, 0, 0};
                    for (int k = 0; k < m; ++k) r[k] = reg(ks);
                    int M = new_match(m, MATCH_INT, ks);
                    for (int k = 0; k < m; ++k) {
                        Cont Kk{2, M, k};
                        cps(s, ops[k], Kk);
                    }
                    // numbered after the call sites inside its arguments, as in the literal graph
                    int label = new_label(callee, K);
                    emit(ks, VM_CALL, r[2], r[0], r[1], label);
                    emit(ks, VM_HALT);
                }
                break;
            }
            case RDF_OP_IF: {
                // the Switch where the predicate arrives: in this segment when it waits for nothing, else in the code
                // that runs when the call it waits for has returned (data-dependent control: which calls fire next is
                // decided by a value a callee computed)
                const rdf_expr xi = x;
                auto branch = [this, xi, K](int s2, int c) {
                    std::map<int, int> saved = segs[s2].memo;
                    size_t brz = segs[s2].code.size();
                    emit(s2, VM_BRZ, 0, c);
                    cps(s2, xi.b, K);
                    size_t jmp = segs[s2].code.size();
                    emit(s2, VM_JMP);
                    segs[s2].memo = saved;
                    segs[s2].code[brz].imm = (int32_t)segs[s2].code.size();
                    cps(s2, xi.c, K);
                    segs[s2].code[jmp].imm = (int32_t)segs[s2].code.size();
                    segs[s2].memo = saved;
                };
                if (call_free(f, x.a)) {
                    branch(s, value(s, x.a));
                } else {
                    Cont Kc{3};
                    Kc.fn = branch;
                    cps(s, x.a, Kc);
                }
                break;
            }
            case RDF_OP_NODE_LOSS: {
                // identity on the state; the invocation's node index must be the parameter
                require(P.ex(f, x.b).op == RDF_OP_PARAM, RDF_ERR_UNSUPPORTED);
                g->has_loss = true;
                cps(s, x.a, K);
                break;
            }
            case RDF_OP_EMBED: case RDF_OP_LEAF_LSTM: {
                require(call_free(f, x.a), RDF_ERR_UNSUPPORTED);
                g->has_vector_ops = true;
                (x.op == RDF_OP_EMBED ? g->has_rnn : g->has_lstm) = true;
                int r = value(s, x.a);
                int ks = cont_segment(K);
                emit(s, x.op == RDF_OP_EMBED ? VM_EMBED : VM_LEAF_LSTM, 0, r, 0, -(ks + 1));   // fixed up at layout
                break;
            }
            case RDF_OP_CHILD_L: case RDF_OP_CHILD_R: {
                g->has_vector_ops = true;
                g->has_rnn = true;
                g->interleaved = true;
                int r = value(s, x.a);
                int ks = cont_segment(K);
                emit(s, VM_VCHILD, x.op == RDF_OP_CHILD_L ? 0 : 1, r, 0, -(ks + 1));            // fixed up at layout
                break;
            }
            case RDF_OP_CELL_RNN: case RDF_OP_CELL_LSTM: {
                g->has_vector_ops = true;
                (x.op == RDF_OP_CELL_RNN ? g->has_rnn : g->has_lstm) = true;
                int ks = cont_segment(K);
                int M = new_match(2, x.op == RDF_OP_CELL_RNN ? MATCH_CELL_RNN : MATCH_CELL_LSTM, ks);
                Cont Ka{2, M, 0}, Kb{2, M, 1};
                cps(s, x.a, Ka);
                cps(s, x.b, Kb);
                break;
            }
            default: {
                // integer operator with at least one operand that depends on a call
                const int ops[2] = {x.a, x.b};
                const uint8_t vop = vm_binop(x.op);
                bool dyn[2];
                int n_dyn = 0;
                for (int k = 0; k < 2; ++k) {
                    dyn[k] = P.ex(f, ops[k]).op != RDF_OP_CONST;
                    n_dyn += dyn[k];
                }
                if (n_dyn == 1) {
                    // one tagged input: no match needed, the operator runs when that input arrives
                    const int kd = dyn[0] ? 0 : 1;
                    const int64_t cv = P.ex(f, ops[1 - kd]).imm;
                    Cont K2{3};
                    K2.fn = [this, vop, kd, cv, K](int s2, int r) {
                        int c = load_const(s2, cv);
                        int d = reg(s2);
                        emit(s2, vop, d, kd == 0 ? r : c, kd == 0 ? c : r);
                        apply(K, s2, d);
                    };
                    cps(s, ops[kd], K2);
                } else {
                    // two tagged inputs meet in the token store; the continuation gets them as r0, r1
                    int ks = new_seg();
                    int r0 = reg(ks), r1 = reg(ks), d = reg(ks);
                    emit(ks, vop, d, r0, r1);
                    apply(K, ks, d);
                    emit(ks, VM_HALT);
                    int M = new_match(2, MATCH_INT, ks);
                    Cont Ka{2, M, 0}, Kb{2, M, 1};
                    cps(s, x.a, Ka);
                    cps(s, x.b, Kb);
                }
            }
        }
    }

    void run() {
        const int nf = P.p->n_functions;
        entry_seg.assign(nf, -1);
        local_count.assign(nf, 0);
        for (int f = 0; f < nf; ++f) {
            entry_seg[f] = new_seg();
            segs[entry_seg[f]].entry = true;
            segs[entry_seg[f]].nregs = std::max(1, P.fn(f).n_params);
        }
        std::vector<int> order{P.p->result};
        for (int f = 0; f < nf; ++f)
            if (f != P.p->result && !P.is_loop(f)) order.push_back(f);          // (loops are lowered where they stand)
        for (int f : order) {
            cur_func = f;
            calls_in_body = 0;
            g->max_params = std::max(g->max_params, P.fn(f).n_params);
            for (int k = 1; k < P.fn(f).n_params; ++k) emit(entry_seg[f], VM_LDARG, k, 0, 0, k);   // parameter k from the frame
            Cont K{f == P.p->result ? 1 : 0};
            cps(entry_seg[f], P.fn(f).root, K);
            emit(entry_seg[f], VM_HALT);
            g->max_calls_per_body = std::max(g->max_calls_per_body, calls_in_body);
        }
        // pairs of calls: a Call_i followed in straight-line code (register moves, arithmetic, tree accessors, parameter
        // loads) by another one -- the two calls of a binary recursion -- reserve their frames and queue slots together
        for (Seg& S : segs)
            for (size_t i = 0; i < S.code.size(); ++i) {
                if (S.code[i].op != VM_CALL) continue;
                for (size_t j = i + 1; j < S.code.size(); ++j) {
                    const uint8_t op = S.code[j].op;
                    if (op == VM_CALL) {
                        S.code[i].op = VM_CALL_A;
                        S.code[j].op = VM_CALL_B;
                        i = j;
                        break;
                    }
                    const bool pure = op == VM_MOVI || op == VM_MOVC || op == VM_MOV || (op >= VM_ADD && op <= VM_REM) ||
                                      op == VM_ISLEAF || op == VM_LEFT || op == VM_RIGHT || op == VM_TOK || op == VM_LDARG;
                    if (!pure) break;
                }
            }
        // layout: concatenate segments, make jump targets absolute
        int pc = 0;
        for (Seg& S : segs) {
            S.base = pc;
            pc += (int)S.code.size();
        }
        require(pc <= RDF_MAX_CODE, RDF_ERR_UNSUPPORTED);
        for (Seg& S : segs)
            for (VmInstr in : S.code) {
                if (in.op == VM_BRZ || in.op == VM_JMP) in.imm += S.base;
                if (in.op == VM_EMBED || in.op == VM_LEAF_LSTM || in.op == VM_VCHILD || in.op == VM_ENTER || in.op == VM_NEXT) in.imm = segs[-in.imm - 1].base;
                g->code.push_back(in);
            }
        for (size_t i = 0; i < g->labels.size(); ++i) {
            g->labels[i].entry_pc = segs[label_entry_seg[i]].base;
            if (label_kseg[i] >= 0) g->labels[i].k_pc = segs[label_kseg[i]].base;
        }
        for (size_t i = 0; i < g->match.size(); ++i) g->match[i].cont_pc = segs[match_cont_seg[i]].base;
        g->result_entry_pc = segs[entry_seg[P.p->result]].base;
        int bits = 1;
        while ((1 << bits) < (int)g->labels.size()) ++bits;
        g->label_bits = bits;
        for (const LabelInfo& L : g->labels) {
            g->label_callee.push_back(L.callee);
            g->label_local.push_back(L.local_label);
        }
        if (g->has_vector_ops) require(P.p->tag_mode == RDF_TAGS_FRAME, RDF_ERR_UNSUPPORTED);
        require(!(g->has_vector_ops && g->has_loops), RDF_ERR_UNSUPPORTED);      // loops are integer programs here
        require(!(g->has_rnn && g->has_lstm), RDF_ERR_UNSUPPORTED);
    }
};

}  // namespace

extern "C" int rdf_graph_build(const rdf_program* prog, rdf_graph** out_graph) {
    if (!prog || !out_graph) return RDF_ERR_BAD_ARG;
    *out_graph = nullptr;
    rdf_graph* g = new rdf_graph();
    try {
        Prog P{prog};
        validate(P);
        check_kinds(P);
        g->tag_mode = prog->tag_mode;
        for (int f = 0; f < prog->n_functions; ++f) g->func_names.push_back(prog->functions[f].name);
        build_literal(P, g);
        Lower L{P, g};
        L.run();
    } catch (const Err& e) {
        delete g;
        return e.code;
    } catch (...) {
        delete g;
        return RDF_ERR_BAD_PROGRAM;
    }
    *out_graph = g;
    return RDF_OK;
}

extern "C" void rdf_graph_free(rdf_graph* g) {
    if (!g) return;
    rdf_exec_release(g);
    delete g;
}

extern "C" int rdf_graph_describe(const rdf_graph* g, rdf_graph_desc* out) {
    if (!g || !out) return RDF_ERR_BAD_ARG;
    out->n_nodes = (int32_t)g->nodes.size();
    out->n_edges = (int32_t)g->edges.size();
    out->nodes = g->nodes.data();
    out->edges = g->edges.data();
    out->n_labels = (int32_t)g->labels.size();
    out->label_bits = g->label_bits;
    out->n_match = (int32_t)g->match.size();
    out->n_code = (int32_t)g->code.size();
    out->label_callee = g->label_callee.data();
    out->label_local = g->label_local.data();
    return RDF_OK;
}

extern "C" const char* rdf_strerror(int status) {
    switch (status) {
        case RDF_OK: return "ok";
        case RDF_ERR_BAD_PROGRAM: return "malformed program";
        case RDF_ERR_BAD_ARG: return "bad argument";
        case RDF_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case RDF_ERR_TAG_OVERFLOW: return "call depth exceeds the packed tag";
        case RDF_ERR_STORE_FULL: return "token store full";
        case RDF_ERR_FRAMES_FULL: return "more invocations than max_invocations";
        case RDF_ERR_QUEUE_FULL: return "wave queue full";
        case RDF_ERR_WAVE_LIMIT: return "wave limit reached (recursion without base case?)";
        case RDF_ERR_TIMEOUT: return "bounded device wait expired";
        case RDF_ERR_CUDA: return "CUDA runtime error";
        case RDF_ERR_UNSUPPORTED: return "program not supported by the device executor";
        default: return "unknown status";
    }
}
