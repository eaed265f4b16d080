// Device executor, forward: persistent, cooperatively launched kernels run all
// waves of the tagged dataflow graph without returning to the host.
//   Scheduler kernel: every wave takes its tokens, runs their segments (tag
//      push / pop, Switch, token-store insert or match) and emits the next
//      wave's tokens.  A vector value travels by reference (the frame that
//      holds it), so a ready leaf / cell operator is queued, not computed: the
//      kernel leaves behind the lists of ready operators, each cell with the
//      height of the operator tree below it.
//   Operator kernel: fires the ready operators as batches, the leaves first and
//      then the cells height by height (grouped by three small kernels between
//      the two): operands before results, in as few dependent waves as possible.
#include <algorithm>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <type_traits>

#include "rdf_exec.h"
#include "rdf_lists.cuh"
#include "rdf_lstm.cuh"
#include "rdf_tc.cuh"

// ===========================================================================
// S phase: the segment interpreter
// ===========================================================================
struct SharedProgram {
    VmInstr   code[RDF_MAX_CODE];
    MatchNode match[RDF_MAX_MATCH];
    LabelInfo labels[RDF_MAX_LABELS];
    int64_t   consts[RDF_MAX_CONSTS];
};

struct ThreadStats {
    uint32_t invocations = 0, tokens = 0, cells = 0, leaves = 0, max_depth = 0, max_height = 0;
    StoreCounters sc;
};

__device__ __forceinline__ void load_program(const DevCtx& c, SharedProgram& sp) {
    for (int i = threadIdx.x; i < c.n_code; i += blockDim.x) sp.code[i] = c.code[i];
    for (int i = threadIdx.x; i < c.n_match; i += blockDim.x) sp.match[i] = c.match[i];
    for (int i = threadIdx.x; i < c.n_labels; i += blockDim.x) sp.labels[i] = c.labels[i];
    for (int i = threadIdx.x; i < c.n_consts; i += blockDim.x) sp.consts[i] = c.consts[i];
    __syncthreads();
}

// A completed match of a batched (cell) operator: queue the cell and the token
// that carries its state onwards in the next wave.
__device__ __forceinline__ void fire_cell(const DevCtx& c, const LocalQ* lq, const MatchNode& M, uint32_t wave, uint64_t tag,
                                          const int64_t* regs, ThreadStats& st) {
    // (global queue: the place in the list and the queue slot of the token that carries the state on are reserved together)
    uint32_t i, slot = 0;
    if (lq) i = aggregated_inc(&lq->ctr[LQ_CELLS]);
    else aggregated_inc2(&c.ctl->cell_count.v, &c.ctl->qcount[(wave + 1) % 3].v, i, slot);
    if (i >= c.work_cap || (!lq && slot >= c.qcap)) {
        set_status(c, RDF_ERR_QUEUE_FULL);
        return;
    }
    // A vector value travels as the frame that holds it (low half of the datum) and the height of the
    // operator tree below it (high half): leaves 0, a cell one more than the higher of its operands.
    CellItem it;
    it.out = (uint32_t)tag; it.l = (uint32_t)regs[0]; it.r = (uint32_t)regs[1];
    it.height = max((uint32_t)((uint64_t)regs[0] >> 32), (uint32_t)((uint64_t)regs[1] >> 32)) + 1u;
    c.cell_items[i] = it;
    st.max_height = max(st.max_height, it.height);
    c.op_l[tag] = it.l;
    c.op_r[tag] = it.r;
    ++st.cells;
    const int64_t datum = (int64_t)(((uint64_t)it.height << 32) | (uint32_t)tag);
    if (lq) push_token(c, lq, wave, tag, datum, (uint32_t)M.cont_pc);
    else store_token(&c.q[(wave + 1) & 1][slot], tag, datum, (uint32_t)M.cont_pc);
}

// Runs one token through its segment and on through every continuation it
// completes (a returning value that finds its partner in the store carries on
// in the caller's context in the same thread).
__device__ void run_token(const DevCtx& c, const SharedProgram& sp, const LocalQ* lq, uint32_t wave, Token t, ThreadStats& st) {
    int64_t r[RDF_MAX_REGS];
    uint64_t tag = t.tag;
    int pc = (int)t.pc;
    r[0] = t.datum;
    ++st.tokens;
    int64_t node_v = -1;                          // tree accessors: the node whose words are in node_l / node_r / node_t
    int32_t node_l = 0, node_r = 0, node_t = 0;
    bool have_pair = false;                       // VM_CALL_A reserved a frame and a queue slot for the VM_CALL_B that follows
    uint32_t pair_id = 0, pair_slot = 0;
    // One instruction per iteration; the bound only guards against a corrupted program.
    for (uint32_t step = 0; step < (1u << 22); ++step) {
        const VmInstr in = sp.code[pc++];
        switch (in.op) {
            case VM_MOVI: r[in.dst] = in.imm; break;
            case VM_MOVC: r[in.dst] = sp.consts[in.imm]; break;
            case VM_MOV: r[in.dst] = r[in.a]; break;
            case VM_ADD: r[in.dst] = r[in.a] + r[in.b]; break;
            case VM_SUB: r[in.dst] = r[in.a] - r[in.b]; break;
            case VM_MUL: r[in.dst] = r[in.a] * r[in.b]; break;
            case VM_MAX: r[in.dst] = r[in.a] > r[in.b] ? r[in.a] : r[in.b]; break;
            case VM_REM: r[in.dst] = r[in.b] == 0 ? 0 : r[in.a] % r[in.b]; break;
            case VM_LT: r[in.dst] = r[in.a] < r[in.b]; break;
            case VM_EQ: r[in.dst] = r[in.a] == r[in.b]; break;
            case VM_ISLEAF: case VM_LEFT: case VM_RIGHT: case VM_TOK: {
                // accessors of the caller's flat tree arrays: an index outside [0, N) is the caller's mistake and
                // ends the token with a status code, never with an access
                const int64_t v = r[in.a];
                if (v < 0 || v >= c.N) {
                    set_status(c, RDF_ERR_BAD_ARG);
                    return;
                }
                // the three words of a node are fetched together the first time one of them is asked for: a body reads
                // is_leaf, then the token or the two children of the same node, and the later reads find their word on its way
                if (v != node_v) {
                    node_v = v;
                    node_l = __ldg(&c.left[v]);
                    if (c.right) node_r = __ldg(&c.right[v]);
                    if (c.tok) node_t = __ldg(&c.tok[v]);
                }
                const int32_t x = in.op == VM_RIGHT ? node_r : in.op == VM_TOK ? node_t : node_l;
                r[in.dst] = in.op == VM_ISLEAF ? (int64_t)(x < 0) : (int64_t)x;
                break;
            }
            case VM_BRZ: if (r[in.a] == 0) pc = in.imm; break;     // Switch: the false side
            case VM_JMP: pc = in.imm; break;
            case VM_CALL: case VM_CALL_A: case VM_CALL_B: {         // Call_i
                uint64_t nt;
                // global queue: the new frame's id (frame-form tags) and the token's queue slot are reserved together, and
                // for a pair of calls (VM_CALL_A .. VM_CALL_B) both calls' places at once
                const bool frames = c.tag_mode != RDF_TAGS_PATH;
                const bool fused = lq == nullptr && (frames || in.op != VM_CALL);
                uint32_t slot = 0, id = 0;
                if (fused) {
                    if (in.op == VM_CALL_B && have_pair) {
                        id = pair_id; slot = pair_slot;
                        have_pair = false;
                    } else if (in.op == VM_CALL_A) {
                        aggregated_inc2n(frames ? &c.ctl->frame_count.v : nullptr, &c.ctl->qcount[(wave + 1) % 3].v, 2u, id, slot);
                        pair_id = id + 1u; pair_slot = slot + 1u;
                        have_pair = true;
                        if (frames && pair_id >= c.frame_cap) {
                            set_status(c, RDF_ERR_FRAMES_FULL);
                            return;
                        }
                    } else aggregated_inc2n(frames ? &c.ctl->frame_count.v : nullptr, &c.ctl->qcount[(wave + 1) % 3].v, 1u, id, slot);
                }
                if (fused && frames) {
                    if (id >= c.frame_cap) {
                        set_status(c, RDF_ERR_FRAMES_FULL);
                        return;
                    }
                    frame_init(c, sp.labels, tag, (uint32_t)in.imm, r[in.a], id, wave);
                    nt = id;
                } else if (!tag_push(c, sp.labels, tag, (uint32_t)in.imm, r[in.a], nt, wave, lq)) return;
                ++st.invocations;
                if (c.tag_mode == RDF_TAGS_PATH) {
                    const uint32_t d = (uint32_t)(nt >> RDF_DEPTH_SHIFT) & 63u;
                    if (d > st.max_depth) st.max_depth = d;
                }
                if (sp.labels[in.imm].n_args > 1) {             // the other Call_i nodes of this call site
                    c.frame_args[(size_t)frame_of(nt) * 2] = r[in.b];
                    c.frame_args[(size_t)frame_of(nt) * 2 + 1] = r[in.dst];
                }
                if (fused) {
                    if (slot >= c.qcap) {
                        set_status(c, RDF_ERR_QUEUE_FULL);
                        return;
                    }
                    store_token(&c.q[(wave + 1) & 1][slot], nt, r[in.a], (uint32_t)sp.labels[in.imm].entry_pc);
                } else push_token(c, lq, wave, nt, r[in.a], (uint32_t)sp.labels[in.imm].entry_pc);
                break;
            }
            case VM_LDARG:                                          // parameter imm of this invocation, from its frame
                r[in.dst] = in.imm == 0 ? __ldcg(reinterpret_cast<const long long*>(&c.frames[frame_of(tag)].arg))
                                        : __ldcg(reinterpret_cast<const long long*>(&c.frame_args[(size_t)frame_of(tag) * 2 + in.imm - 1]));
                break;
            case VM_ENTER: {                                        // Enter: <t, d> -> <0:t, d>
                // a loop frame under the current tag: counter 0 in the high half of the new tag, the tag below kept whole
                const uint32_t id = aggregated_inc(lq ? &lq->ctr[LQ_FRAMES] : &c.ctl->frame_count.v);
                if (id >= c.frame_cap) {
                    set_status(c, RDF_ERR_FRAMES_FULL);
                    return;
                }
                Frame f;
                f.parent = frame_of(tag); f.label = LOOP_LABEL | (wave << FRAME_WAVE_SHIFT); f.arg = r[in.a];
                c.frames[id] = f;
                c.frame_ptag[id] = tag;
                c.frame_args[(size_t)id * 2] = r[in.b];             // variables 1 and 2 live in the loop frame
                c.frame_args[(size_t)id * 2 + 1] = r[in.dst];
                trace_rec(c, id, r[in.a], 2, LOOP_LABEL, tag);
                push_token(c, lq, wave, (uint64_t)id, r[in.a], (uint32_t)in.imm);
                break;
            }
            case VM_NEXT: {                                         // Next: <n:t, d> -> <(n+1):t, d>
                const int64_t v0 = r[in.a], v1 = r[in.b], v2 = r[in.dst];
                c.frame_args[(size_t)frame_of(tag) * 2] = v1;
                c.frame_args[(size_t)frame_of(tag) * 2 + 1] = v2;
                const uint64_t nt = tag + (1ull << 32);
                trace_rec(c, nt, v0, 3, LOOP_LABEL, 0);
                push_token(c, lq, wave, nt, v0, (uint32_t)in.imm);
                return;                                             // this iteration's token ends here
            }
            case VM_EXIT: {                                         // Exit: <n:t, d> -> <t, d>
                trace_rec(c, tag, r[in.a], 4, LOOP_LABEL, 0);
                tag = __ldcg(reinterpret_cast<const unsigned long long*>(&c.frame_ptag[frame_of(tag)]));
                break;
            }
            case VM_RET:
            case VM_PORT: {
                const int64_t val = r[in.a];
                int node = -1, port = 0;
                if (in.op == VM_PORT) {
                    node = in.imm;
                    port = in.b;
                } else {
                    // Return_i: pop until the value reaches an operator of some caller
                    for (;;) {
                        uint32_t label;
                        uint64_t parent;
                        tag_pop(c, tag, label, parent);
                        trace_rec(c, tag, c.H > 0 ? (int64_t)(uint32_t)val : val, 1, label, parent);   // (vector value: its frame)
                        tag = parent;
                        const LabelInfo& L = sp.labels[label];
                        if (L.k_kind == K_RET) continue;           // the call was the caller's own output
                        if (L.k_kind == K_SEG) {
                            r[0] = val;
                            pc = L.k_pc;
                        } else {
                            node = L.k_node;
                            port = L.k_port;
                        }
                        break;
                    }
                    if (node < 0) break;                            // continue in the caller's segment
                }
                const MatchNode& M = sp.match[node];
                int done;
                if (c.tag_mode == RDF_TAGS_PATH) {
                    int64_t partner = 0;
                    done = c.probe_mode ? hash_insert_or_consume_group(c, node, tag, val, partner, st.sc)
                                        : hash_insert_or_consume(c, node, tag, val, partner, st.sc);
                    if (done < 0) {
                        set_status(c, RDF_ERR_STORE_FULL);
                        return;
                    }
                    if (done) {
                        r[port] = val;
                        r[1 - port] = partner;
                    }
                } else {
                    done = dense_deliver(c, M, node, tag, port, val, r, st.sc);
                }
                if (!done) {
                    if (in.op == VM_RET) return;                    // parked: this token's journey ends here
                    break;                                          // VM_PORT inside a segment: carry on
                }
                if (M.kind == MATCH_INT) {
                    pc = M.cont_pc;                                 // r[0..n) hold the operands
                    break;
                }
                fire_cell(c, lq, M, wave, tag, r, st);
                return;
            }
            case VM_OUT: {
                const long long inst = c.tag_mode == RDF_TAGS_PATH ? (long long)(tag >> RDF_INST_SHIFT) : (long long)tag;
                if (inst >= 0 && inst < c.B) c.y[inst] = c.H > 0 ? (int64_t)(uint32_t)r[in.a] : r[in.a];   // (vector value: its frame)
                return;
            }
            case VM_EMBED:
            case VM_LEAF_LSTM: {
                if (r[in.a] < 0 || r[in.a] >= c.V) {             // a token id that is no row of the embedding table
                    set_status(c, RDF_ERR_BAD_ARG);
                    return;
                }
                uint32_t i, slot = 0;
                if (lq) i = aggregated_inc(&lq->ctr[LQ_LEAVES]);
                else aggregated_inc2(&c.ctl->leaf_count.v, &c.ctl->qcount[(wave + 1) % 3].v, i, slot);
                if (i >= c.work_cap || (!lq && slot >= c.qcap)) {
                    set_status(c, RDF_ERR_QUEUE_FULL);
                    return;
                }
                LeafItem it;
                it.slot = (uint32_t)tag;
                it.tok = (int32_t)r[in.a];
                c.leaf_items[i] = it;
                c.op_l[tag] = LEAF_MARK;
                c.op_r[tag] = (uint32_t)it.tok;
                ++st.leaves;
                if (lq) push_token(c, lq, wave, tag, (int64_t)tag, (uint32_t)in.imm);
                else store_token(&c.q[(wave + 1) & 1][slot], tag, (int64_t)tag, (uint32_t)in.imm);
                break;
            }
            case VM_VGATE: {
                // An integer read off a vector value: W_s[0] . h + b_s[0] > 0 in fp32, terms added in index order.  The
                // state was written by the operator phase of an earlier wave (any block): read through L2.
                const uint32_t ref = (uint32_t)r[in.a];
                if (ref >= c.frame_cap) {
                    set_status(c, RDF_ERR_BAD_ARG);
                    return;
                }
                const float* h = c.arena + (size_t)ref * c.S;
                float acc = c.b_s[0];
                for (int k = 0; k < c.H; ++k) acc = fmaf(__ldg(&c.W_s[k]), __ldcg(&h[k]), acc);
                r[in.dst] = acc > 0.f;
                break;
            }
            case VM_VCHILD: {
                // a unary vector operator: queued like a cell whose second operand is the marker of the operator
                uint32_t i, slot = 0;
                aggregated_inc2(&c.ctl->cell_count.v, &c.ctl->qcount[(wave + 1) % 3].v, i, slot);
                if (i >= c.work_cap || slot >= c.qcap) {
                    set_status(c, RDF_ERR_QUEUE_FULL);
                    return;
                }
                CellItem it;
                it.out = (uint32_t)tag; it.l = (uint32_t)r[in.a]; it.r = in.dst ? CHILD_R_MARK : CHILD_L_MARK;
                it.height = (uint32_t)((uint64_t)r[in.a] >> 32) + 1u;
                c.cell_items[i] = it;
                st.max_height = max(st.max_height, it.height);
                c.op_l[tag] = it.l;
                c.op_r[tag] = it.r;
                ++st.cells;
                store_token(&c.q[(wave + 1) & 1][slot], tag, (int64_t)(((uint64_t)it.height << 32) | (uint32_t)tag), (uint32_t)in.imm);
                break;
            }
            default:   // VM_HALT
                return;
        }
    }
    set_status(c, RDF_ERR_WAVE_LIMIT);
}

// ===========================================================================
// C phase, fp32: leaf gather and the TreeRNN cell as a tiled FFMA contraction
// ===========================================================================
// out[i][j] = tanh( sum_k W[j][k] * x_i[k] + b[j] ),  x_i = [state(l_i) ; state(r_i)]
__device__ void rnn_cell_tiles(const DevCtx& c, GemmSmem& sm, uint32_t first, uint32_t n_items) {
    const int H = c.H, K2 = 2 * c.H;
    const int tiles_m = (n_items + TM - 1) / TM, tiles_n = (H + TN - 1) / TN;
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
    const int lrow = threadIdx.x / 4, lk = (threadIdx.x % 4) * 4;
    for (int tile = blockIdx.x; tile < tiles_m * tiles_n; tile += gridDim.x) {
        const int tm = tile / tiles_n, tn = tile % tiles_n;
        const int row0 = tm * TM, col0 = tn * TN;
        // this thread's source rows for the operand loads
        const int arow = row0 + lrow;
        const float *xl = nullptr, *xr = nullptr;
        if (arow < (int)n_items) {
            const uint4 it = __ldcg(reinterpret_cast<const uint4*>(&c.cell_items[first + arow]));   // {out, l, r, -}
            xl = c.arena + (size_t)it.y * H;
            xr = c.arena + (size_t)it.z * H;
        }
        const int bcol = col0 + lrow;
        const float* wrow = bcol < H ? c.W + (size_t)bcol * K2 : nullptr;
        float acc[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
        // the operands of step k0 + TK are on their way (registers) while step k0 is multiplied
        auto fetch = [&](int k0, float4& a, float4& b) {
            const int k = k0 + lk;
            a = make_float4(0.f, 0.f, 0.f, 0.f); b = a;
            if (xl && k < K2) a = k < H ? ldcg4(xl + k) : ldcg4(xr + (k - H));
            if (wrow && k < K2) b = __ldg(reinterpret_cast<const float4*>(wrow + k));
        };
        float4 a, b;
        fetch(0, a, b);
        for (int k0 = 0; k0 < K2; k0 += TK) {
            __syncthreads();
            sm.As[lk + 0][lrow] = a.x; sm.As[lk + 1][lrow] = a.y; sm.As[lk + 2][lrow] = a.z; sm.As[lk + 3][lrow] = a.w;
            sm.Bs[lk + 0][lrow] = b.x; sm.Bs[lk + 1][lrow] = b.y; sm.Bs[lk + 2][lrow] = b.z; sm.Bs[lk + 3][lrow] = b.w;
            __syncthreads();
            if (k0 + TK < K2) fetch(k0 + TK, a, b);
            gemm_tile_step(sm, tx, ty, acc);
        }
        const int col = col0 + tx * 4;
        if (col < H) {
            const float4 bias = __ldg(reinterpret_cast<const float4*>(c.b + col));
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int row = row0 + ty * 4 + i;
                if (row < (int)n_items) {
                    const uint32_t out = __ldcg(&c.cell_items[first + row].out);
                    float4 v;
                    v.x = tanhf(acc[i][0] + bias.x); v.y = tanhf(acc[i][1] + bias.y);
                    v.z = tanhf(acc[i][2] + bias.z); v.w = tanhf(acc[i][3] + bias.w);
                    *reinterpret_cast<float4*>(c.arena + (size_t)out * H + col) = v;
                }
            }
        }
    }
}

// Narrow waves (a few dozen ready cells, e.g. the tail of a deep chain): the 64 x 64 tiles would keep
// a handful of blocks busy with a long dependent k-loop.  Here one block step computes an 8 cell x 16
// column patch with the whole contraction spread over its threads: thread = (cell, column, half of k),
// streaming its operand row and weight row with independent 128-bit loads.
// wres: this block's resident 16 columns of W in shared memory (or nullptr), as float4 [k / 4][column]:
// the 16 columns of the column group blockIdx.x % units_n, which is the group of every patch the block
// gets while a wave has no more patches than blocks.
__device__ void rnn_cell_thin(const DevCtx& c, float* xs, const float4* wres, uint32_t first, uint32_t n_items) {
    // xs: shared staging for the 8 operand rows [h_l ; h_r] of the patch (8 x 2H floats) + 128 floats
    const int H = c.H, K2 = 2 * c.H;
    float* red = xs + 8 * K2;
    const int units_n = (H + 15) / 16, units = ((n_items + 7) / 8) * units_n;
    const int o = threadIdx.x & 127, kh = threadIdx.x >> 7, rr = o >> 4, cc = o & 15;
    for (int unit = blockIdx.x; unit < units; unit += gridDim.x) {
        const int row0 = (unit / units_n) * 8;
        // all operand rows of the patch in one round of independent 128-bit loads
        for (int p = threadIdx.x; p < 8 * (K2 / 4); p += blockDim.x) {
            const int r = p / (K2 / 4), k = (p % (K2 / 4)) * 4;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (row0 + r < (int)n_items) {
                const uint4 it = __ldcg(reinterpret_cast<const uint4*>(&c.cell_items[first + row0 + r]));   // {out, l, r, -}
                v = k < H ? ldcg4(c.arena + (size_t)it.y * H + k) : ldcg4(c.arena + (size_t)it.z * H + (k - H));
            }
            *reinterpret_cast<float4*>(xs + r * K2 + k) = v;
        }
        __syncthreads();
        const int row = row0 + rr, col = (unit % units_n) * 16 + cc;
        const bool live = row < (int)n_items && col < H;
        float acc = 0.f;
        if (live) {
            const float4* x = reinterpret_cast<const float4*>(xs + rr * K2 + kh * H);
            float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
            if (wres && unit % units_n == (int)(blockIdx.x % units_n)) {
                const float4* w = wres + (size_t)(kh * (H / 4)) * 16 + cc;          // lanes: consecutive columns, no bank conflicts
#pragma unroll 8
                for (int k4 = 0; k4 < H / 4; ++k4) {
                    const float4 xv = x[k4], wv = w[k4 * 16];
                    a0 = fmaf(xv.x, wv.x, a0); a1 = fmaf(xv.y, wv.y, a1);
                    a2 = fmaf(xv.z, wv.z, a2); a3 = fmaf(xv.w, wv.w, a3);
                }
            } else {
                const float4* w = reinterpret_cast<const float4*>(c.W + (size_t)col * K2 + kh * H);
#pragma unroll 8
                for (int k4 = 0; k4 < H / 4; ++k4) {
                    const float4 xv = x[k4], wv = __ldg(w + k4);
                    a0 = fmaf(xv.x, wv.x, a0); a1 = fmaf(xv.y, wv.y, a1);
                    a2 = fmaf(xv.z, wv.z, a2); a3 = fmaf(xv.w, wv.w, a3);
                }
            }
            acc = (a0 + a1) + (a2 + a3);
        }
        if (kh == 1) red[o] = acc;
        __syncthreads();
        if (kh == 0 && live)
            c.arena[(size_t)__ldcg(&c.cell_items[first + row].out) * H + col] = tanhf(acc + red[o] + __ldg(&c.b[col]));
        __syncthreads();
    }
}

__device__ void rnn_leaf_rows(const DevCtx& c, uint32_t n_items) {
    // one warp per leaf: state(slot) = E[tok]
    const int H = c.H;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) / 32, lane = threadIdx.x % 32;
    const int n_warps = gridDim.x * blockDim.x / 32;
    for (uint32_t i = warp; i < n_items; i += n_warps) {
        const uint2 it = __ldcg(reinterpret_cast<const uint2*>(&c.leaf_items[i]));          // {slot, tok}
        const float4* src = reinterpret_cast<const float4*>(c.E + (size_t)it.y * c.D);
        float4* dst = reinterpret_cast<float4*>(c.arena + (size_t)it.x * H);
        for (int k = lane; k < H / 4; k += 32) dst[k] = __ldg(src + k);
    }
}

// ===========================================================================
// the persistent forward kernel
// ===========================================================================
// per-thread counters -> one set of atomics per warp
__device__ __forceinline__ void flush_stats(const DevCtx& c, const ThreadStats& st) {
    unsigned long long v[7] = {st.invocations, st.tokens, st.cells, st.leaves, st.sc.inserts, st.sc.matches, st.sc.probes};
    uint32_t mp = st.sc.max_probe, md = st.max_depth, mh = st.max_height;
    for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
        for (int k = 0; k < 7; ++k) v[k] += __shfl_xor_sync(0xffffffffu, v[k], o);
        mp = max(mp, __shfl_xor_sync(0xffffffffu, mp, o));
        md = max(md, __shfl_xor_sync(0xffffffffu, md, o));
        mh = max(mh, __shfl_xor_sync(0xffffffffu, mh, o));
    }
    if ((threadIdx.x & 31) == 0) {
        atomicAdd(&c.ctl->invocations, v[0]); atomicAdd(&c.ctl->tokens, v[1]); atomicAdd(&c.ctl->cells, v[2]);
        atomicAdd(&c.ctl->leaves, v[3]); atomicAdd(&c.ctl->store_inserts, v[4]); atomicAdd(&c.ctl->store_matches, v[5]);
        atomicAdd(&c.ctl->store_probes, v[6]);
        atomicMax(&c.ctl->max_probe, mp);
        atomicMax(&c.ctl->max_depth, md);
        if (mh) atomicMax(&c.ctl->max_height, mh);        // (the operator waves run height by height)
    }
}

static const uint32_t NARROW_STRETCH = 4096;   // waves block 0 runs alone before it meets the grid again

// The scheduler: all waves of token processing, for integer and for vector programs.  Only tokens are
// handled here, so the block is 1024 threads wide: the dependent L2 round trips of a token (queue,
// frame table, store) are hidden by the number of tokens in flight.
__global__ void __launch_bounds__(1024, 1) rdf_scheduler_kernel(const __grid_constant__ DevCtx c) {
    __shared__ SharedProgram sp;
    __shared__ uint32_t lq_count[3], lq_ctr[3];
    extern __shared__ __align__(16) unsigned char lq_smem[];         // local queue of narrow stretches: 2 x LQ_CAP tokens
    LocalQ lq;
    lq.buf[0] = reinterpret_cast<Token*>(lq_smem);
    lq.buf[1] = lq.buf[0] + LQ_CAP;
    lq.count = lq_count;
    lq.ctr = lq_ctr;
    load_program(c, sp);
    ThreadStats st;
    uint32_t generation = 0, wave = 0, widest = 0;
    long long cyc_s = 0, cyc_b = 0, t_mark = clock64();
    auto lap = [&](long long& acc) {
        const long long now = clock64();
        acc += now - t_mark;
        t_mark = now;
    };
    for (;; ++wave) {
        // the thread's first token of the wave is fetched together with the wave's token count (a slot past the count
        // holds an old token, which is dropped)
        const uint32_t gi = blockIdx.x * blockDim.x + threadIdx.x;
        const Token first_tok = gi < c.qcap ? load_token(&c.q[wave & 1][gi]) : Token{};
        const uint32_t n = ld_volatile_u32(&c.ctl->qcount[wave % 3].v);
        if (n == 0) break;
        if (wave >= c.wave_limit) {
            set_status(c, RDF_ERR_WAVE_LIMIT);
            break;
        }
        widest = max(widest, n);
        if (n <= blockDim.x) {
            // A stretch of narrow waves (deep, thin recursion): one block has a thread for every token,
            // so block 0 runs wave after wave with a block barrier between them while the other blocks
            // wait at the grid barrier below.  It comes back to the grid when a wave is wider than the
            // block, when the queue is empty, or after NARROW_STRETCH waves (so that the bounded
            // wait of the other blocks never expires on a long stretch).
            if (blockIdx.x == 0) {
                // The tokens of the stretch stay in this block's shared memory: the first wave is read from
                // the global queue, the following ones from the local queue, and what is left at the end
                // goes back to the global queue.
                uint32_t m = n, k = 0;
                bool local = false;
                if (threadIdx.x < 3) lq_count[threadIdx.x] = 0;
                // the other blocks are on their way to the grid barrier and reserve nothing: this block owns the counters
                if (threadIdx.x == 0) {
                    lq_ctr[LQ_FRAMES] = ld_volatile_u32(&c.ctl->frame_count.v);
                    lq_ctr[LQ_CELLS] = ld_volatile_u32(&c.ctl->cell_count.v);
                    lq_ctr[LQ_LEAVES] = ld_volatile_u32(&c.ctl->leaf_count.v);
                }
                __syncthreads();
                do {
                    if (threadIdx.x == 0) lq_count[(wave + 2) % 3] = 0;
                    if (threadIdx.x < m) {
                        const Token t = local ? load_local_token(&lq.buf[wave & 1][threadIdx.x]) : first_tok;   // (block 0: gi == threadIdx.x)
                        run_token(c, sp, &lq, wave, t, st);
                    }
                    __syncthreads();          // orders this wave's queue writes before the next wave's reads (same block)
                    if (k == 0) {
                        // The end of the stretch rewrites the counters that the other blocks read to take this
                        // branch: carry on only when all of them have arrived at the grid barrier below (they
                        // read the counter before they arrive).  Bounded like every other wait.
                        __shared__ int others_in;
                        if (threadIdx.x == 0) {
                            const uint32_t target = generation * gridDim.x + gridDim.x - 1;
                            const long long t0 = clock64();
                            int good = 1;
                            while (ld_volatile_u32(&c.ctl->bar.v) < target) {
                                if (clock64() - t0 > c.spin_limit) {
                                    set_status(c, RDF_ERR_TIMEOUT);
                                    good = 0;
                                    break;
                                }
                                if (ld_volatile_i32(&c.ctl->status) != 0) {       // another block gave up: so does this one
                                    good = 0;
                                    break;
                                }
                            }
                            others_in = good;
                        }
                        __syncthreads();
                        if (!others_in) {
                            ++wave;
                            m = 0;
                            break;
                        }
                    }
                    ++wave;
                    ++k;
                    local = true;
                    m = lq_count[wave % 3];
                    widest = max(widest, m);
                } while (m != 0 && m <= blockDim.x && k < NARROW_STRETCH && wave < c.wave_limit &&
                         ld_volatile_i32(&c.ctl->status) == 0);
                // hand the next wave back to the global queue (tokens beyond the local capacity are there already)
                for (uint32_t i = threadIdx.x; i < min(m, LQ_CAP); i += blockDim.x) {
                    const Token t = load_local_token(&lq.buf[wave & 1][i]);
                    store_token(&c.q[wave & 1][i], t.tag, t.datum, t.pc);
                }
                if (threadIdx.x == 0) {
                    c.ctl->qcount[wave % 3].v = m;
                    c.ctl->qcount[(wave + 1) % 3].v = 0;
                    c.ctl->resume_wave = wave;
                    c.ctl->frame_count.v = lq_ctr[LQ_FRAMES];
                    c.ctl->cell_count.v = lq_ctr[LQ_CELLS];
                    c.ctl->leaf_count.v = lq_ctr[LQ_LEAVES];
                }
            }
            lap(cyc_s);
            if (!grid_barrier(c, &c.ctl->bar.v, generation)) break;
            lap(cyc_b);
            wave = ld_volatile_u32(&c.ctl->resume_wave) - 1;      // the loop header adds the one back
            continue;
        }
        if (blockIdx.x == 0 && threadIdx.x == 0) c.ctl->qcount[(wave + 2) % 3].v = 0;
        const Token* q = c.q[wave & 1];
        {
            // a wave wider than the grid: the thread's next token is on its way while it runs the current one
            const uint32_t stride = gridDim.x * blockDim.x;
            uint32_t i = gi;
            Token next = first_tok;
            while (i < n) {
                const Token cur = next;
                i += stride;
                if (i < n) next = load_token(&q[i]);
                run_token(c, sp, nullptr, wave, cur, st);
            }
        }
        __syncthreads();
        lap(cyc_s);
        if (!grid_barrier(c, &c.ctl->bar.v, generation)) break;
        lap(cyc_b);
    }
    flush_stats(c, st);
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        c.ctl->waves = wave;
        c.ctl->max_wave_tokens = widest;
        c.ctl->cyc[0] = cyc_s; c.ctl->cyc[2] = cyc_b;
        c.ctl->forward_status = c.ctl->status;      // what the operator kernel checks before it starts
    }
}


static inline int interleaved_smem_bytes(int H) { return 2 * H * 33 * (int)sizeof(float); }

// Token scheduling and vector operators interleaved wave by wave, for programs in which a Switch reads a vector
// value (RDF_OP_GATE): the tokens of wave w may read any state whose operator was queued before wave w, so every
// wave ends with the operators it queued -- leaves E[tok], unary operators tanh(W_half x + b), cells
// tanh(W [x_l ; x_r] + b) -- in groups of 32 operators per block.
// Two grid barriers per wave (tokens | operators).  fp32, H <= INTERLEAVED_MAX_H.
__global__ void __launch_bounds__(1024, 1) rdf_interleaved_kernel(const __grid_constant__ DevCtx c) {
    __shared__ SharedProgram sp;
    extern __shared__ __align__(16) unsigned char il_smem[];
    load_program(c, sp);
    ThreadStats st;
    uint32_t generation = 0, wave = 0, widest = 0, done_cells = 0, done_leaves = 0;
    long long cyc_s = 0, cyc_o = 0, cyc_b = 0, t_mark = clock64();
    auto lap = [&](long long& acc) {
        const long long now = clock64();
        acc += now - t_mark;
        t_mark = now;
    };
    const int H = c.H, lane = threadIdx.x % 32, warp = threadIdx.x / 32;
    float* xs = reinterpret_cast<float*>(il_smem);                  // [2H][33]: operand rows of a group of 32 operators, transposed
    const uint32_t gwarp = blockIdx.x * (blockDim.x / 32) + warp, n_warps = gridDim.x * (blockDim.x / 32);
    for (;; ++wave) {
        const uint32_t n = ld_volatile_u32(&c.ctl->qcount[wave % 3].v);
        if (n == 0) break;
        if (wave >= c.wave_limit) {
            set_status(c, RDF_ERR_WAVE_LIMIT);
            break;
        }
        widest = max(widest, n);
        if (blockIdx.x == 0 && threadIdx.x == 0) c.ctl->qcount[(wave + 2) % 3].v = 0;
        const Token* q = c.q[wave & 1];
        for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x)
            run_token(c, sp, nullptr, wave, load_token(&q[i]), st);
        __syncthreads();
        lap(cyc_s);
        if (!grid_barrier(c, &c.ctl->bar.v, generation)) break;
        lap(cyc_b);
        // ---- the operators this wave queued
        const uint32_t n_leaf = min(ld_volatile_u32(&c.ctl->leaf_count.v), c.work_cap);
        const uint32_t n_cell = min(ld_volatile_u32(&c.ctl->cell_count.v), c.work_cap);
        for (uint32_t i = done_leaves + gwarp; i < n_leaf; i += n_warps) {
            const LeafItem it = c.leaf_items[i];
            const float* e = c.E + (size_t)it.tok * c.D;
            float* out = c.arena + (size_t)it.slot * c.S;
            for (int k = lane; k < H; k += 32) out[k] = __ldg(&e[k]);
        }
        // Unary operators and cells, 32 at a time per block: a unary operator on x is the cell on [x ; 0] (left half of
        // W) or [0 ; x] (right half), so one loop serves all three.  The operand rows of the group are staged
        // transposed (xs[k][item], rows padded to 33 floats: conflict-free both ways); warp w then computes outputs
        // 4w .. 4w+3 (+128, ...) of all 32 items, lane = item, the weight rows read as uniform vector loads.
        for (uint32_t g0 = done_cells + blockIdx.x * 32u; g0 < n_cell; g0 += gridDim.x * 32u) {
            const uint32_t cnt = min(32u, n_cell - g0);
            __syncthreads();                                        // (the previous group's operands are no longer read)
            CellItem it = CellItem{0u, 0u, 0u, 0u};
            bool ok = false;
            if ((uint32_t)warp < cnt) {
                it = c.cell_items[g0 + warp];
                const bool unary = it.r == CHILD_L_MARK || it.r == CHILD_R_MARK;
                ok = it.l < c.frame_cap && (unary || it.r < c.frame_cap) && it.out < c.frame_cap;
                if (!ok && lane == 0) set_status(c, RDF_ERR_BAD_ARG);
                for (int k = lane; k < H; k += 32) {
                    float a = 0.f, b2 = 0.f;
                    if (ok) {
                        const float x = __ldcg(&c.arena[(size_t)it.l * c.S + k]);
                        if (it.r == CHILD_R_MARK) b2 = x; else a = x;
                        if (!unary) b2 = __ldcg(&c.arena[(size_t)it.r * c.S + k]);
                    }
                    xs[(size_t)k * 33 + warp] = a;
                    xs[(size_t)(H + k) * 33 + warp] = b2;
                }
            }
            __syncthreads();
            // lane = item of the group; its output row
            const uint32_t out_row = (uint32_t)lane < cnt ? c.cell_items[g0 + lane].out : 0xFFFFFFFFu;
            for (int j0 = warp * 4; j0 < H; j0 += 128) {
                float acc[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) acc[q] = c.b[j0 + q];
                const float4* w0 = reinterpret_cast<const float4*>(c.W + (size_t)j0 * 2 * H);
                const int K4 = 2 * H / 4;
                for (int k4 = 0; k4 < K4; ++k4) {
                    float4 w[4];
#pragma unroll
                    for (int q = 0; q < 4; ++q) w[q] = __ldg(w0 + (size_t)q * K4 + k4);
                    const float x0 = xs[(size_t)(4 * k4 + 0) * 33 + lane], x1 = xs[(size_t)(4 * k4 + 1) * 33 + lane];
                    const float x2 = xs[(size_t)(4 * k4 + 2) * 33 + lane], x3 = xs[(size_t)(4 * k4 + 3) * 33 + lane];
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        acc[q] = fmaf(w[q].w, x3, fmaf(w[q].z, x2, fmaf(w[q].y, x1, fmaf(w[q].x, x0, acc[q]))));
                }
                if (out_row < c.frame_cap)
                    *reinterpret_cast<float4*>(c.arena + (size_t)out_row * c.S + j0) =
                        make_float4(tanhf(acc[0]), tanhf(acc[1]), tanhf(acc[2]), tanhf(acc[3]));
            }
        }
        done_leaves = n_leaf;
        done_cells = n_cell;
        __syncthreads();
        lap(cyc_o);
        if (!grid_barrier(c, &c.ctl->bar.v, generation)) break;
        lap(cyc_b);
    }
    flush_stats(c, st);
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        c.ctl->waves = wave;
        c.ctl->max_wave_tokens = widest;
        c.ctl->cyc[0] = cyc_s; c.ctl->cyc[1] = cyc_o; c.ctl->cyc[2] = cyc_b;
        c.ctl->forward_status = c.ctl->status;
    }
}

__global__ void __launch_bounds__(256) rdf_seed_kernel(const DevCtx c) {
    const long long b = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= c.B) return;
    // one token <[], x_b> per instance enters `result`
    uint64_t tag;
    const int64_t datum = c.x ? c.x[b] : (int64_t)c.tree_root[b];
    if (c.tag_mode == RDF_TAGS_PATH) {
        tag = path_root(b);
    } else {
        tag = (uint64_t)b;            // frames 0..B-1 are the contexts of `result`
        Frame f;
        f.parent = LEAF_MARK; f.label = 0; f.arg = datum;          // (wave field 0: before the first wave)
        c.frames[b] = f;
        if (c.finst) c.finst[b] = (uint32_t)b;
    }
    store_token(&c.q[0][b], tag, datum, (uint32_t)c.result_entry_pc);
    if (b == 0) {
        c.ctl->qcount[0].v = (uint32_t)c.B;
        c.ctl->frame_count.v = c.tag_mode == RDF_TAGS_FRAME ? (uint32_t)c.B : 0u;
    }
}

// The operator kernel: the leaves first (they wait for nothing), then the cells in waves whose operands are complete;
// a grid barrier separates the waves.  fp32 FMA tiles: height by height (a cell reads states of smaller heights).
// TC: bf16 operands on the tensor cores (the tile pipeline of rdf_tc.cuh), depth by depth from the deepest cells up.
// RNN32: the fp32 TreeRNN alone (no TreeLSTM code in the kernel): few enough registers for two blocks per SM, which is what
// the FFMA tiles need to hide their shared-memory and barrier latencies.
template <bool TC, bool RNN32 = false>
__global__ void __launch_bounds__(TC ? TC_THREADS : 256, RNN32 ? 2 : 1) rdf_operator_kernel(const __grid_constant__ DevCtx c) {
    __shared__ typename std::conditional<TC, TcShared, LstmSmem>::type smem;   // (the TreeRNN tiles and patches use the first part of LstmSmem)
    const bool lstm = RNN32 ? false : c.lstm != 0;
    extern __shared__ unsigned char dyn_smem[];                      // TC: resident weight slices + operand stages
    if (c.ctl->forward_status != 0) return;                          // the scheduler failed: the lists are not to be trusted
    TcState tc;
    if constexpr (TC) {
        if (lstm) tc_setup(tc, smem, dyn_smem, c.Hp / 16, c.Wp, 2 * c.Hp, 80, c.Wxp, c.Hp, 48);
        else tc_setup(tc, smem, dyn_smem, 4, c.Wp, 2 * c.Hp, c.Hp / 4);
        tc_setup_epilogue(c, tc, smem, false);
    }
    // fp32 TreeRNN, narrow waves: this block's 16 columns of W stay in shared memory for all waves
    const float4* wres = nullptr;
    if constexpr (!TC) {
        if (!lstm && c.H <= THIN_RESIDENT_MAX_H) {
            float4* wr = reinterpret_cast<float4*>(dyn_smem);
            const int K2 = 2 * c.H, units_n = (c.H + 15) / 16, cg0 = blockIdx.x % units_n;
            for (int q = threadIdx.x; q < (K2 / 4) * 16; q += blockDim.x) {
                const int k4 = q / 16, col = cg0 * 16 + q % 16;
                wr[q] = col < c.H ? __ldg(reinterpret_cast<const float4*>(c.W + (size_t)col * K2) + k4) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
            __syncthreads();
            wres = wr;
        }
    }
    uint32_t generation = 0;
    long long cyc_c = 0, cyc_b = 0, t_mark = clock64();
    auto lap = [&](long long& acc) {
        const long long now = clock64();
        acc += now - t_mark;
        t_mark = now;
    };
    const uint32_t n_leaf = min(c.ctl->leaf_count.v, c.work_cap);
    bool alive = true;
    if (n_leaf) {
        if constexpr (TC) {
            if (lstm) tc_pipe<TC_LSTM_LEAF, TC_STAGES_LSTM_FWD>(c, tc, smem, 0, n_leaf);
            else {
                tc_leaf_rows(c, n_leaf);
                asm volatile("fence.proxy.async;" ::: "memory");      // the operand rows it wrote are read by tile copies after the barrier
            }
        } else {
            if constexpr (RNN32) rnn_leaf_rows(c, n_leaf);
            else {
                if (lstm) lstm_forward_tiles<3>(c, smem, 0, n_leaf);
                else rnn_leaf_rows(c, n_leaf);
            }
        }
        __syncthreads();
        lap(cyc_c);
        alive = grid_barrier(c, &c.ctl->bar_ops.v, generation);
        lap(cyc_b);
    }
    if constexpr (TC) {
        // Tensor-core path: the cells depth by depth, deepest first (the states a cell of depth k reads belong to
        // depth k + 1).  The cells of one depth are consecutive in the cell list, and so are their operand rows,
        // which their callees wrote: the tiles read plain 2D boxes.
        const uint32_t nw = min(c.ctl->n_depth_waves, c.wave_cap);
        uint4 wv = nw ? c.wave_marks[nw - 1] : make_uint4(0u, 0u, 0u, 0u);      // {first frame, end frame, first cell, end cell}
        for (uint32_t k = nw; k-- > 0 && alive;) {
            const uint4 cur = wv;
            if (k > 0) wv = c.wave_marks[k - 1];                         // in flight during this wave
            if (cur.w <= cur.z) continue;                                // (a depth of leaves only)
            const uint32_t first = min(cur.z, c.cells_cap), nc = min(cur.w, c.cells_cap) - first;
            if (lstm) tc_pipe<TC_LSTM_CELL, TC_STAGES_LSTM_FWD>(c, tc, smem, first, nc);
            else tc_pipe<TC_RNN_FWD, TC_STAGES_RNN_FWD>(c, tc, smem, first, nc);
            __syncthreads();
            lap(cyc_c);
            alive = grid_barrier(c, &c.ctl->bar_ops.v, generation);
            lap(cyc_b);
        }
    } else {
        // fp32 path: height by height (cell_items is the sorted list here: the launch passes cell_sorted in its place).
        // With the clustered path the list is sorted by (group of instances, height): this kernel fires the wide heights
        // (1 .. h_split: every group's cells of the height, then one barrier) and leaves the rest to the clusters.
        const uint32_t groups = cell_groups(c), stride = min(c.ctl->max_height, c.wave_cap) + 1u;
        const uint32_t top = groups > 1u ? min(c.ctl->h_split, stride - 1u) : stride - 1u;
        for (uint32_t w = 1; w <= top && alive; ++w) {
            bool any = false;
            for (uint32_t gq = 0; gq < groups; ++gq) {
                const uint32_t first = min(c.height_ends[(size_t)gq * stride + w - 1], c.work_cap);
                const uint32_t end = min(c.height_ends[(size_t)gq * stride + w], c.work_cap);
                if (end <= first) continue;                              // (no cell of this height in the group)
                const uint32_t nc = end - first;
                any = true;
                bool done = false;
                if constexpr (!RNN32) {
                    if (lstm) {
                        lstm_forward_tiles<5>(c, smem, first, nc);
                        done = true;
                    }
                }
                // thin patches while they fit in two rounds over the grid, tiles for wide waves
                if (done) {
                } else if (c.H <= 384 && ((nc + 7) / 8) * ((c.H + 15) / 16) <= 2 * gridDim.x)
                    rnn_cell_thin(c, reinterpret_cast<float*>(&smem), wres, first, nc);      // 8 x 2H + 128 floats <= 26 KB
                else rnn_cell_tiles(c, *reinterpret_cast<GemmSmem*>(&smem), first, nc);
                __syncthreads();
            }
            if (!any) continue;
            lap(cyc_c);
            alive = grid_barrier(c, &c.ctl->bar_ops.v, generation);
            lap(cyc_b);
        }
    }
    if constexpr (TC) tc_teardown(tc);
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        c.ctl->cyc[1] = cyc_c;
        c.ctl->cyc[2] += cyc_b;
    }
}

// ===========================================================================
// fp32 TreeRNN cells without a grid barrier: one thread-block cluster per group of instances
// ===========================================================================
// Tokens of different instances never meet (matching needs equal tags, and a tag belongs to one instance), so the cells
// of different instances do not depend on one another.  The ready cells are sorted by (group of their instance,
// height); a cluster of CLUSTER_CTAS blocks fires the cells of its group height by height and synchronises with the
// hardware cluster barrier only -- a deep, thin recursion (a wave of a few dozen cells, thousands of waves) pays about
// a microsecond per wave instead of a barrier over the whole grid.  The blocks of a cluster split the columns of W
// (kept in shared memory for the whole kernel); a block step computes `cells_per_step` cells x its columns, thread =
// (cell, column), operand rows staged in shared memory.  States travel between the blocks through global memory
// (L2): the cluster barrier's release / acquire orders them.

// CPC: columns of W per block (8 blocks x CPC >= H).  A block step fires CS = 256 / CPC cells: thread = (column, slice
// of the contraction index), CS accumulators per thread -- a weight is read from shared memory once per step and an
// operand word once per warp; the slices are added up through shared memory by thread = (cell, column).
template <int CPC>
__global__ void __launch_bounds__(256, 1) rdf_operator_cluster_kernel(const __grid_constant__ DevCtx c) {
    constexpr int CS = 256 / CPC;              // cells per step = slices of k
    extern __shared__ __align__(16) unsigned char dyn_smem[];
    // every block of the grid takes the same decision from the same words: no block of a cluster is left waiting
    if (c.ctl->forward_status != 0 || cell_groups(c) <= 1u) return;
    const int H = c.H, K2 = 2 * c.H;
    const int rank = blockIdx.x % CLUSTER_CTAS, group = blockIdx.x / CLUSTER_CTAS;
    const int j0 = rank * CPC;
    float* wres = reinterpret_cast<float*>(dyn_smem);                  // [K2][CPC]: this block's columns of W
    float* xs = wres + (size_t)K2 * CPC;                               // [2][CS][K2]: operand rows, double buffered
    float* part = xs + (size_t)2 * CS * K2;                            // [CS slices][CS cells][CPC]: partial sums
    uint32_t* s_out = reinterpret_cast<uint32_t*>(part + (size_t)CS * CS * CPC);   // [2][CS]: frames of the results
    for (int q = threadIdx.x; q < K2 * CPC; q += blockDim.x) {
        const int k = q / CPC, jj = q % CPC;
        wres[q] = j0 + jj < H ? __ldg(&c.W[(size_t)(j0 + jj) * K2 + k]) : 0.f;
    }
    __syncthreads();
    const uint32_t stride = min(c.ctl->max_height, c.wave_cap) + 1u, top = stride - 1u;
    const uint32_t* ends = c.height_ends + (size_t)group * stride;      // ends[h]: end of (group, h); ends[0]: start of the group
    const int jj = threadIdx.x % CPC, ks = threadIdx.x / CPC;           // column; slice of k (contraction) / cell (reduction)
    const bool active = ks < CS;
    const int klen = ((K2 + CS - 1) / CS + 3) & ~3, k_begin = ks * klen, k_end = min(K2, k_begin + klen);
    const float bias = active && j0 + jj < H ? __ldg(&c.b[j0 + jj]) : 0.f;
    // rows of a step: CS cells x K2 floats, fetched by all threads as 128-bit pieces
    const int pieces = CS * (K2 / 4);
    // (pre: the records of the step's cells when they were fetched ahead -- thread p holds the record of row p / (K2 / 4)
    //  of its first piece -- else null)
    auto stage = [&](int buf, uint32_t first, uint32_t n, const uint4* pre) {
        float* dst = xs + (size_t)buf * CS * K2;
        for (int p = threadIdx.x; p < pieces; p += blockDim.x) {
            const int r = p / (K2 / 4), k = (p % (K2 / 4)) * 4;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if ((uint32_t)r < n) {
                const uint4 it = pre && p == (int)threadIdx.x ? *pre : __ldcg(reinterpret_cast<const uint4*>(&c.cell_items[first + r]));   // {out, l, r, height}
                v = k < H ? ldcg4(c.arena + (size_t)it.y * H + k) : ldcg4(c.arena + (size_t)it.z * H + (k - H));
                if (k == 0) s_out[buf * CS + r] = it.x;
            }
            *reinterpret_cast<float4*>(dst + (size_t)r * K2 + k) = v;
        }
    };
    const uint32_t h0 = min(c.ctl->h_split, top);                     // (the grid-wide kernel fired heights 1 .. h0)
    uint32_t begin = min(ends[h0], c.work_cap);
    uint32_t end_next = top > h0 ? min(ends[h0 + 1], c.work_cap) : begin;
    // the list is complete before the kernel starts: the record this thread needs first in the next wave is fetched a wave ahead
    const int my_row = threadIdx.x / (K2 / 4);
    uint4 rec_next = make_uint4(0u, 0u, 0u, 0u);
    if (threadIdx.x < pieces && begin + my_row < end_next) rec_next = __ldcg(reinterpret_cast<const uint4*>(&c.cell_items[begin + my_row]));
    for (uint32_t h = h0 + 1; h <= top; ++h) {
        const uint32_t end = end_next;
        if (h < top) end_next = min(ends[h + 1], c.work_cap);           // in flight during this wave
        // the cells of (group, h), CS at a time; the next step's rows are fetched while this one computes
        int buf = 0;
        const uint4 rec = rec_next;
        if (end > begin) stage(0, begin, min((uint32_t)CS, end - begin), &rec);
        if (threadIdx.x < pieces && end + my_row < end_next) rec_next = __ldcg(reinterpret_cast<const uint4*>(&c.cell_items[end + my_row]));
        for (uint32_t first = begin; first < end; first += CS) {
            const uint32_t n = min((uint32_t)CS, end - first);
            __syncthreads();                                            // rows of this step are in place, `part` is free
            if (first + CS < end) stage(buf ^ 1, first + CS, min((uint32_t)CS, end - first - CS), nullptr);
            if (active) {
                float acc[CS];
#pragma unroll
                for (int q = 0; q < CS; ++q) acc[q] = 0.f;
                const float* x = xs + (size_t)buf * CS * K2;
                for (int k = k_begin; k < k_end; k += 4) {
                    const float w0 = wres[(size_t)k * CPC + jj], w1 = wres[(size_t)(k + 1) * CPC + jj];
                    const float w2 = wres[(size_t)(k + 2) * CPC + jj], w3 = wres[(size_t)(k + 3) * CPC + jj];
#pragma unroll
                    for (int q = 0; q < CS; ++q) {
                        const float4 xv = *reinterpret_cast<const float4*>(x + (size_t)q * K2 + k);   // (one word for the whole warp)
                        acc[q] = fmaf(xv.x, w0, fmaf(xv.y, w1, fmaf(xv.z, w2, fmaf(xv.w, w3, acc[q]))));
                    }
                }
#pragma unroll
                for (int q = 0; q < CS; ++q) part[((size_t)ks * CS + q) * CPC + jj] = acc[q];
            }
            __syncthreads();
            if (active && (uint32_t)ks < n && j0 + jj < H) {            // thread = (cell ks, column jj): the slices added in order
                float t = bias;
#pragma unroll
                for (int q = 0; q < CS; ++q) t += part[((size_t)q * CS + ks) * CPC + jj];
                c.arena[(size_t)s_out[buf * CS + ks] * H + j0 + jj] = tanhf(t);
            }
            buf ^= 1;
        }
        begin = end;
        __syncthreads();
        cluster_sync_all();                                             // the states of height h are complete for the whole cluster
    }
}

inline int cluster_cols_per_block(int H) { return H <= 64 ? 8 : H <= 128 ? 16 : H <= 256 ? 32 : 48; }
inline size_t cluster_smem_bytes(int H) {
    const int CPC = cluster_cols_per_block(H), CS = 256 / CPC, K2 = 2 * H;
    return ((size_t)K2 * CPC + (size_t)2 * CS * K2 + (size_t)CS * CS * CPC) * sizeof(float) + 2 * CS * sizeof(uint32_t);
}
static const int CLUSTER_MAX_H = 384;

// ---- cells grouped by height (between the scheduler and the operator kernel)
// The scheduler finds a cell ready in the wave in which its second operand returns, which depends on how deep the
// whole tree below it reaches; what the arithmetic needs is only that operands come first.  Grouping the cells by
// height gives the smallest number of dependent operator waves (the largest height instead of about twice the depth).
// (With the clustered operator kernel the cells are grouped by (cluster of their instance, height): bucket index
// group * (max height + 1) + height; one group otherwise.  The largest height is known from the scheduler.)
__device__ __forceinline__ uint32_t cell_bucket(const DevCtx& c, const CellItem& it, uint32_t groups, uint32_t stride, int by_depth) {
    if (it.height == 0u) return 0u;                                                  // (0: not a cell)
    // by_depth (gradient pass): the scheduler wave that created the cell's frame, + 1
    const uint32_t h = min(by_depth ? (__ldcg(&c.frames[it.out].label) >> FRAME_WAVE_SHIFT) + 1u : it.height, stride - 1u);
    return (groups > 1u ? __ldcg(&c.finst[it.out]) % groups : 0u) * stride + h;
}

__global__ void __launch_bounds__(256) rdf_height_count_kernel(const DevCtx c, int by_depth) {
    if (c.ctl->status != 0) return;
    const uint32_t n = min(c.ctl->cell_count.v, c.work_cap), lane = threadIdx.x % 32;
    const uint32_t groups = bucket_groups(c, by_depth), stride = bucket_stride(c, by_depth);
    for (uint32_t i0 = (blockIdx.x * blockDim.x + threadIdx.x) & ~31u; i0 < n; i0 += gridDim.x * blockDim.x) {
        const uint32_t i = i0 + lane;
        const uint32_t k = i < n ? cell_bucket(c, c.cell_items[i], groups, stride, by_depth) : 0u;
        const unsigned peers = __match_any_sync(0xffffffffu, k);                      // one atomic per bucket and warp
        if (k && (uint32_t)(__ffs(peers) - 1) == lane) atomicAdd(&c.height_ends[k], (uint32_t)__popc(peers));
    }
}

// counts -> first position of each bucket (one block; buckets 1 .. groups * (max height + 1) - 1)
__global__ void __launch_bounds__(1024) rdf_height_scan_kernel(const DevCtx c, int by_depth) {
    __shared__ uint32_t warp_sum[32];
    __shared__ uint32_t carry;
    if (c.ctl->status != 0) return;
    const uint32_t top = bucket_groups(c, by_depth) * bucket_stride(c, by_depth) - 1u;
    const uint32_t lane = threadIdx.x % 32, warp = threadIdx.x / 32;
    if (threadIdx.x == 0) carry = 0;
    __syncthreads();
    for (uint32_t h0 = 1; h0 <= top; h0 += 1024) {
        const uint32_t h = h0 + threadIdx.x;
        const uint32_t v = h <= top ? c.height_ends[h] : 0u;
        uint32_t x = v;
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t y = __shfl_up_sync(0xffffffffu, x, o);
            if ((int)lane >= o) x += y;
        }
        if (lane == 31) warp_sum[warp] = x;
        __syncthreads();
        if (warp == 0) {
            uint32_t w = warp_sum[lane];
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t y = __shfl_up_sync(0xffffffffu, w, o);
                if ((int)lane >= o) w += y;
            }
            warp_sum[lane] = w;
        }
        __syncthreads();
        const uint32_t before = carry + (warp ? warp_sum[warp - 1] : 0u) + x - v;
        if (h <= top) c.height_ends[h] = before;
        __syncthreads();
        if (threadIdx.x == 1023) carry = before + v;
        __syncthreads();
    }
}

// every cell to its bucket; afterwards height_ends[k] is where bucket k ends (it starts where bucket k - 1 ends;
// bucket group * stride + 0 is empty, so it ends where the previous group ends)
__global__ void __launch_bounds__(256) rdf_height_scatter_kernel(const DevCtx c, int by_depth) {
    if (c.ctl->status != 0) return;
    const uint32_t n = min(c.ctl->cell_count.v, c.work_cap), lane = threadIdx.x % 32;
    const uint32_t groups = bucket_groups(c, by_depth), stride = bucket_stride(c, by_depth);
    for (uint32_t i0 = (blockIdx.x * blockDim.x + threadIdx.x) & ~31u; i0 < n; i0 += gridDim.x * blockDim.x) {
        const uint32_t i = i0 + lane;
        CellItem it = i < n ? c.cell_items[i] : CellItem{0u, 0u, 0u, 0u};
        const uint32_t k = cell_bucket(c, it, groups, stride, by_depth);
        const unsigned peers = __match_any_sync(0xffffffffu, k);
        const int leader = __ffs(peers) - 1;
        uint32_t base = 0;
        if (k && (uint32_t)leader == lane) base = atomicAdd(&c.height_ends[k], (uint32_t)__popc(peers));
        base = __shfl_sync(0xffffffffu, base, leader);
        if (k) c.cell_sorted[min(base + (uint32_t)__popc(peers & ((1u << lane) - 1u)), c.work_cap - 1u)] = it;
    }
}

// Which heights are wide enough for the whole grid (clustered path): the last height that has more than `threshold` cells
// over all groups; the heights above it are left to the clusters.
__global__ void __launch_bounds__(256) rdf_height_split_kernel(const DevCtx c, uint32_t threshold, int by_depth) {
    if (c.ctl->status != 0) return;
    const uint32_t groups = bucket_groups(c, by_depth), stride = bucket_stride(c, by_depth);
    if (groups <= 1u) return;
    for (uint32_t h = 1 + blockIdx.x * blockDim.x + threadIdx.x; h < stride; h += gridDim.x * blockDim.x) {
        uint32_t total = 0;
        for (uint32_t gq = 0; gq < groups; ++gq) total += c.height_ends[(size_t)gq * stride + h] - c.height_ends[(size_t)gq * stride + h - 1];
        if (total > threshold) atomicMax(by_depth ? &c.ctl->d_split : &c.ctl->h_split, h);
    }
}

// root states: h_root[b] = state(frame y[b])
__global__ void rdf_gather_roots_kernel(const DevCtx c, float* h_root) {
    const int b = blockIdx.x;
    const long long slot = c.y[b];
    if (slot < 0 || slot >= (long long)c.frame_cap) return;
    for (int k = threadIdx.x; k < c.H; k += blockDim.x)
        h_root[(size_t)b * c.H + k] = c.arena ? c.arena[(size_t)slot * c.S + k]
                                              : __bfloat162float(c.arena_bf[(size_t)slot * c.Hp + k]);
}

// ===========================================================================
// host side: workspace plan, launches
// ===========================================================================
namespace {

struct Plan {
    size_t off = 0;
    template <class T>
    size_t take(size_t count) {
        off = (off + 255) & ~(size_t)255;
        size_t at = off;
        off += count * sizeof(T);
        return at;
    }
};

uint64_t pow2_at_least(uint64_t v) {
    uint64_t p = 1024;
    while (p < v) p <<= 1;
    return p;
}

}  // namespace

int rdf_make_layout(const rdf_graph* g, const rdf_batch* in, const rdf_params* params, int want_grad, Layout& L) {
    if (!g || !in || in->B <= 0 || in->max_invocations <= 0) return RDF_ERR_BAD_ARG;
    if (g->has_vector_ops && (!params || params->H <= 0 || params->H % 4 != 0)) return RDF_ERR_BAD_ARG;
    if (in->B + in->max_invocations >= 0xFFFFFFF0ll) return RDF_ERR_BAD_ARG;
    if (g->tag_mode == RDF_TAGS_PATH && in->B > (1ll << 20)) return RDF_ERR_BAD_ARG;
    if (want_grad && !g->has_vector_ops) return RDF_ERR_UNSUPPORTED;
    if (g->interleaved) {
        // a Switch reads a vector value: token waves and operators interleaved, fp32, forward only
        if (want_grad || params->compute == RDF_BF16 || params->H > INTERLEAVED_MAX_H || params->D != params->H) return RDF_ERR_UNSUPPORTED;
        if (!params->W_s || !params->b_s || !params->W || !params->b || !params->E) return RDF_ERR_BAD_ARG;
    }
    const int H = g->has_vector_ops ? params->H : 0;
    Plan P;
    L.qcap = (uint32_t)std::min<long long>(in->max_wave_tokens > 0 ? in->max_wave_tokens : in->max_invocations + in->B,
                                           0x7FFFFFFFll);
    L.qcap = std::max<uint32_t>(L.qcap, (uint32_t)in->B);
    L.frame_cap = g->tag_mode == RDF_TAGS_FRAME ? (uint32_t)(in->B + in->max_invocations) : 0;
    L.work_cap = g->has_vector_ops ? L.frame_cap : 0;       // the operator lists hold every invocation of the run
    L.ctl = P.take<char>(4096);
    L.code = P.take<VmInstr>(g->code.size());
    L.match = P.take<MatchNode>(std::max<size_t>(1, g->match.size()));
    L.labels = P.take<LabelInfo>(std::max<size_t>(1, g->labels.size()));
    L.consts = P.take<int64_t>(std::max<size_t>(1, g->consts.size()));
    L.q0 = P.take<Token>(L.qcap);
    L.q1 = P.take<Token>(L.qcap);
    L.frames = P.take<Frame>(L.frame_cap);
    L.frame_args = P.take<int64_t>(g->max_params > 1 || g->has_loops ? (size_t)L.frame_cap * 2 : 0);
    L.frame_ptag = P.take<uint64_t>(g->has_loops ? (size_t)L.frame_cap : 0);
    // fp32 TreeRNN: the cells are fired cluster by cluster of instances (no grid barrier); needs the instance of every frame
    // (eligibility only: whether the device takes clusters is known at launch, and the workspace must not depend on it)
    L.clustered = g->has_vector_ops && g->has_rnn && !g->has_lstm && !g->interleaved && H <= CLUSTER_MAX_H &&
                  !(params->compute == RDF_BF16 && (H + 63) / 64 * 64 <= TC_HP_MAX && params->D == params->H);   // (not the tensor-core path)
    L.finst = P.take<uint32_t>(L.clustered ? (size_t)L.frame_cap : 0);
    L.pair_bytes = (size_t)L.frame_cap * g->match.size() * sizeof(Slot);
    L.pair_slots = P.take<char>(L.pair_bytes);
    L.port_val = P.take<int64_t>((size_t)L.frame_cap * g->n_ports_total);
    L.arrived_bytes = (size_t)L.frame_cap * std::max<size_t>(1, g->match.size()) * sizeof(uint32_t);
    L.arrived = P.take<char>(L.arrived_bytes);
    L.table_cap = g->tag_mode == RDF_TAGS_PATH && !g->match.empty() ? pow2_at_least((uint64_t)in->max_invocations) : 0;
    {
        const ExecState* S = static_cast<const ExecState*>(g->dev);
        if (S && S->hash_slots > 0 && L.table_cap) L.table_cap = pow2_at_least((uint64_t)S->hash_slots);
    }
    L.table_bytes = (size_t)L.table_cap * g->match.size() * sizeof(Slot);
    L.table = P.take<char>(L.table_bytes);
    L.cell_items = P.take<CellItem>(L.work_cap);
    L.leaf_items = P.take<LeafItem>(L.work_cap);
    L.cell_sorted = P.take<CellItem>(g->has_vector_ops ? L.work_cap : 0);
    const size_t vf = g->has_vector_ops ? L.frame_cap : 0;
    L.op_l = P.take<uint32_t>(vf);
    L.op_r = P.take<uint32_t>(vf);
    const size_t S = g->has_lstm ? 2 * (size_t)H : (size_t)H;
    L.Hp = (H + 63) / 64 * 64;
    L.use_tc = g->has_vector_ops && params->compute == RDF_BF16 && L.Hp <= TC_HP_MAX && params->D == params->H;
    const bool tcl = L.use_tc && g->has_lstm, tcr = L.use_tc && !g->has_lstm;
    L.arena = P.take<float>(tcr ? 0 : vf * S);          // the bf16 TreeRNN keeps its states in arena_bf only
    L.gates = P.take<float>(g->has_lstm && want_grad ? vf * 5 * H : 0);
    const size_t wcount = (size_t)L.Hp * 2 * L.Hp * (tcl ? 5 : 1);
    L.arena_bf = P.take<__nv_bfloat16>(L.use_tc ? vf * L.Hp : 0);
    L.wp = P.take<__nv_bfloat16>(L.use_tc ? wcount : 0);
    L.wtp = P.take<__nv_bfloat16>(L.use_tc ? wcount : 0);
    // a cell makes two calls, so a run has at most half as many cells as invocations; rows in whole tiles, one tile to spare
    L.cells_cap = L.use_tc ? ((uint32_t)(vf / 2 + 1) + 127u) / 128u * 128u + 128u : 0;
    L.want_grad = want_grad;
    L.dz_bf = P.take<__nv_bfloat16>(tcr && want_grad ? (size_t)L.cells_cap * L.Hp : 0);
    L.z_bf = P.take<__nv_bfloat16>(L.use_tc ? (size_t)L.cells_cap * 2 * L.Hp : 0);
    L.zdst = P.take<uint32_t>(L.use_tc ? vf : 0);
    L.cell_pos = P.take<uint32_t>(L.use_tc ? vf : 0);
    L.wxp = P.take<__nv_bfloat16>(tcl ? (size_t)3 * L.Hp * L.Hp : 0);
    L.wxtp = P.take<__nv_bfloat16>(tcl ? (size_t)3 * L.Hp * L.Hp : 0);
    L.e_bf = P.take<__nv_bfloat16>(tcl ? (size_t)params->V * L.Hp : 0);
    L.dg_bf = P.take<__nv_bfloat16>(tcl && want_grad ? vf * 5 * L.Hp : 0);
    L.tc_smem_fwd = !L.use_tc ? 0 : tcl ? tc_smem_bytes(80, 2 * L.Hp, 48, L.Hp, TC_STAGES_LSTM_FWD) : tc_smem_bytes(L.Hp / 4, 2 * L.Hp, 0, 0, TC_STAGES_RNN_FWD);
    L.tc_smem_bwd = !L.use_tc ? 0 : tcl ? tc_smem_bytes(TC_LSTM_BWD_NS, 5 * L.Hp, 0, 0, TC_STAGES_LSTM_BWD) : tc_smem_bytes(L.Hp / 4, L.Hp, 0, 0, TC_STAGES_RNN_BWD);
    L.ybuf = P.take<int64_t>(g->has_vector_ops ? in->B : 0);
    const size_t gf = want_grad ? L.frame_cap : 0;
    L.dhp = P.take<float>(tcr ? 0 : gf * S);            // (the bf16 TreeRNN hands its gradients on as dz rows)
    L.dlog = P.take<float>(gf * 8);
    // every wave of a vector program holds at least one token of an invocation on its way down or up
    L.wave_cap = g->has_vector_ops ? (uint32_t)std::min<long long>(2 * (long long)L.frame_cap + 64, 1ll << 24) : 0;
    L.wave_marks = P.take<uint4>(L.wave_cap);
    L.height_ends = P.take<uint32_t>(L.wave_cap ? (size_t)L.wave_cap + 2 : 0);
    // the lists over the frames: the gradient pass needs them, and so do the tensor-core operator waves
    const size_t lf = want_grad || L.use_tc ? L.frame_cap : 0;
    L.list_seg = P.take<uint2>(lf ? (size_t)in->max_invocations / LIST_SEG + 2 : 0);
    L.all_cells = P.take<uint32_t>(lf);
    L.cell_ops = P.take<uint4>(L.use_tc ? lf : 0);
    L.leaf_ops = P.take<uint4>(tcl ? gf : 0);
    L.all_leaves = P.take<uint32_t>(g->has_lstm ? lf : gf);
    L.loss_partial = P.take<float>(want_grad ? 4096 : 0);
    L.repro = want_grad && L.use_tc && params->reproducible ? 1 : 0;
    L.dw_partial = P.take<float>(L.repro ? (size_t)DW_BLOCKS_MAX * 65536 : 0);
    L.de_fix = P.take<long long>(L.repro ? (size_t)params->V * params->D : 0);
    L.head_fix = P.take<long long>(L.repro ? (size_t)params->n_classes * (H + 1) + 1 : 0);
    L.rank_tmp = P.take<uint32_t>(L.repro ? (size_t)2 * L.frame_cap : 0);      // 64-bit keys of the cells or of the leaves
    L.canon_cap = L.repro ? (uint32_t)std::min<unsigned long long>(std::max<unsigned long long>(1ull << 20, 8ull * L.frame_cap), 1ull << 28) : 0;
    L.node_info = P.take<uint2>(L.repro ? (size_t)std::max<long long>(in->N, 1) : 0);
    L.canon_hist = P.take<uint32_t>(L.repro ? (size_t)L.canon_cap + 1 : 0);
    L.total = (P.off + 255) & ~(size_t)255;
    return RDF_OK;
}

ExecState* rdf_state_of(rdf_graph* g) {
    if (!g->dev) g->dev = new ExecState();
    return static_cast<ExecState*>(g->dev);
}

int rdf_prepare_device(rdf_graph* g, ExecState* S) {
    (void)g;
    int dev = 0;
    CUDA_OK(cudaGetDevice(&dev));
    if (S->device == dev && S->grid > 0) return RDF_OK;
    int sms = 0, per_sm = 0, coop = 0;
    CUDA_OK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    CUDA_OK(cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev));
    CUDA_OK(cudaDeviceGetAttribute(&S->clock_khz, cudaDevAttrClockRate, dev));
    if (!coop) return RDF_ERR_CUDA;
    const int max_dyn = std::max(tc_smem_bytes(80, 2 * TC_HP_MAX, 48, TC_HP_MAX, TC_STAGES_LSTM_FWD),
                                 tc_smem_bytes(TC_HP_MAX / 4, 2 * TC_HP_MAX, 0, 0, TC_STAGES_RNN_FWD));   // the largest configurations
    CUDA_OK(cudaFuncSetAttribute(rdf_operator_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_dyn));
    CUDA_OK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, rdf_operator_kernel<true>, TC_THREADS, max_dyn));
    if (per_sm < 1) return RDF_ERR_CUDA;
    CUDA_OK(cudaFuncSetAttribute(rdf_operator_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 128 * THIN_RESIDENT_MAX_H));
    CUDA_OK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, rdf_operator_kernel<false>, 256, 128 * THIN_RESIDENT_MAX_H));
    if (per_sm < 1) return RDF_ERR_CUDA;
    CUDA_OK(cudaFuncSetAttribute(rdf_interleaved_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, interleaved_smem_bytes(INTERLEAVED_MAX_H)));
    CUDA_OK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, rdf_interleaved_kernel, 1024, interleaved_smem_bytes(INTERLEAVED_MAX_H)));
    if (per_sm < 1) return RDF_ERR_CUDA;
    CUDA_OK(cudaFuncSetAttribute(rdf_scheduler_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(2 * LQ_CAP * sizeof(Token))));
    CUDA_OK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, rdf_scheduler_kernel, 1024, 2 * LQ_CAP * sizeof(Token)));
    if (per_sm < 1) return RDF_ERR_CUDA;
    S->grid = sms;                 // one persistent block per SM
    {   // the fp32 TreeRNN kernels: two blocks per SM where they fit
        int a = 0;
        CUDA_OK(cudaFuncSetAttribute(rdf_operator_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 128 * THIN_RESIDENT_MAX_H));
        CUDA_OK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&a, rdf_operator_kernel<false, true>, 256, 128 * THIN_RESIDENT_MAX_H));
        S->rnn32_per_sm = std::max(1, std::min(2, a));
    }
    S->device = dev;
    // the clustered fp32 operator kernel: how many clusters of CLUSTER_CTAS blocks the device holds at once
    S->n_clusters = 0;
    {
        const size_t smem = cluster_smem_bytes(CLUSTER_MAX_H);
        bool ok = cudaFuncSetAttribute(rdf_operator_cluster_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)cluster_smem_bytes(64)) == cudaSuccess &&
                  cudaFuncSetAttribute(rdf_operator_cluster_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)cluster_smem_bytes(128)) == cudaSuccess &&
                  cudaFuncSetAttribute(rdf_operator_cluster_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)cluster_smem_bytes(256)) == cudaSuccess &&
                  cudaFuncSetAttribute(rdf_operator_cluster_kernel<48>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) == cudaSuccess;
        cudaLaunchConfig_t cfg = {};
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = CLUSTER_CTAS; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
        cfg.gridDim = dim3((sms / CLUSTER_CTAS) * CLUSTER_CTAS); cfg.blockDim = dim3(256); cfg.dynamicSmemBytes = smem;
        cfg.attrs = at; cfg.numAttrs = 1;
        int n = 0;
        if (ok && cudaOccupancyMaxActiveClusters(&n, rdf_operator_cluster_kernel<48>, &cfg) == cudaSuccess)
            S->n_clusters = std::min(n, sms / CLUSTER_CTAS);
        else
            cudaGetLastError();            // (no clusters: the grid-wide kernel is used)
    }
    return RDF_OK;
}

void rdf_fill_ctx(rdf_graph* g, const rdf_batch* in, const rdf_params* params, rdf_outputs* out, char* ws,
                  const Layout& L, ExecState* S, DevCtx& c) {
    memset(&c, 0, sizeof(c));
    c.code = reinterpret_cast<const VmInstr*>(ws + L.code);
    c.match = reinterpret_cast<const MatchNode*>(ws + L.match);
    c.labels = reinterpret_cast<const LabelInfo*>(ws + L.labels);
    c.consts = reinterpret_cast<const int64_t*>(ws + L.consts);
    c.n_code = (int)g->code.size(); c.n_match = (int)g->match.size();
    c.n_labels = (int)g->labels.size(); c.n_consts = (int)g->consts.size();
    c.label_bits = g->label_bits; c.tag_mode = g->tag_mode; c.result_entry_pc = g->result_entry_pc;
    c.n_ports_total = g->n_ports_total; c.K = g->max_calls_per_body;
    c.finst = L.clustered ? reinterpret_cast<uint32_t*>(ws + L.finst) : nullptr;
    c.n_groups = L.clustered && S->n_clusters > 1 ? S->n_clusters : 0;
    c.has_loops = g->has_loops ? 1 : 0;
    c.frame_ptag = g->has_loops ? reinterpret_cast<uint64_t*>(ws + L.frame_ptag) : nullptr;
    c.B = in->B; c.N = in->N; c.x = in->x;
    c.tree_root = in->tree_root; c.left = in->left; c.right = in->right; c.tok = in->tok; c.label = in->label;
    c.q[0] = reinterpret_cast<Token*>(ws + L.q0); c.q[1] = reinterpret_cast<Token*>(ws + L.q1);
    c.qcap = L.qcap;
    c.frames = reinterpret_cast<Frame*>(ws + L.frames);
    c.frame_args = reinterpret_cast<int64_t*>(ws + L.frame_args);
    c.frame_cap = L.frame_cap;
    c.pair_slots = reinterpret_cast<Slot*>(ws + L.pair_slots);
    c.port_val = reinterpret_cast<int64_t*>(ws + L.port_val);
    c.arrived = reinterpret_cast<uint32_t*>(ws + L.arrived);
    c.table = reinterpret_cast<Slot*>(ws + L.table);
    c.table_cap = L.table_cap;
    c.cell_items = reinterpret_cast<CellItem*>(ws + L.cell_items);
    c.cell_sorted = reinterpret_cast<CellItem*>(ws + L.cell_sorted);
    c.height_ends = reinterpret_cast<uint32_t*>(ws + L.height_ends);
    c.leaf_items = reinterpret_cast<LeafItem*>(ws + L.leaf_items);
    c.work_cap = L.work_cap;
    c.op_l = reinterpret_cast<uint32_t*>(ws + L.op_l);
    c.op_r = reinterpret_cast<uint32_t*>(ws + L.op_r);
    c.arena = L.use_tc && !g->has_lstm ? nullptr : reinterpret_cast<float*>(ws + L.arena);
    if (g->has_vector_ops) {
        c.H = params->H; c.D = params->D; c.V = params->V; c.n_classes = params->n_classes; c.compute = params->compute;
        c.E = params->E; c.W = params->W; c.b = params->b; c.W_x = params->W_x; c.b_x = params->b_x;
        c.W_s = params->W_s; c.b_s = params->b_s;
        c.y = reinterpret_cast<int64_t*>(ws + L.ybuf);
        c.lstm = g->has_lstm ? 1 : 0;
        c.S = g->has_lstm ? 2 * params->H : params->H;
        c.G = 5 * params->H;
        c.gates = nullptr;                 // set by rdf_grad for the TreeLSTM
        c.use_tc = L.use_tc; c.Hp = L.Hp;
        c.arena_bf = reinterpret_cast<__nv_bfloat16*>(ws + L.arena_bf);
        c.Wp = reinterpret_cast<__nv_bfloat16*>(ws + L.wp);
        c.WTp = reinterpret_cast<__nv_bfloat16*>(ws + L.wtp);
        c.dz_bf = L.use_tc && !g->has_lstm && L.want_grad ? reinterpret_cast<__nv_bfloat16*>(ws + L.dz_bf) : nullptr;
        c.z_bf = L.use_tc ? reinterpret_cast<__nv_bfloat16*>(ws + L.z_bf) : nullptr;
        c.zdst = L.use_tc ? reinterpret_cast<uint32_t*>(ws + L.zdst) : nullptr;
        c.cells_cap = L.cells_cap;
        c.cell_pos = L.use_tc ? reinterpret_cast<uint32_t*>(ws + L.cell_pos) : nullptr;
        c.Wxp = reinterpret_cast<__nv_bfloat16*>(ws + L.wxp);
        c.WxTp = reinterpret_cast<__nv_bfloat16*>(ws + L.wxtp);
        c.E_bf = reinterpret_cast<__nv_bfloat16*>(ws + L.e_bf);
        // only present (and only non-null) for the TreeLSTM on the tensor-core path
        c.dg_bf = L.use_tc && g->has_lstm ? reinterpret_cast<__nv_bfloat16*>(ws + L.dg_bf) : nullptr;
    } else {
        c.y = out->y;
    }
    c.trace = out->trace; c.trace_cap = out->trace ? out->trace_capacity : 0;
    c.dhp = L.use_tc && !g->has_lstm ? nullptr : reinterpret_cast<float*>(ws + L.dhp);
    c.dlog = reinterpret_cast<float*>(ws + L.dlog);
    c.wave_marks = L.wave_cap ? reinterpret_cast<uint4*>(ws + L.wave_marks) : nullptr;
    c.wave_cap = L.wave_cap;
    c.all_cells = reinterpret_cast<uint32_t*>(ws + L.all_cells);
    c.cell_ops = L.use_tc ? reinterpret_cast<uint4*>(ws + L.cell_ops) : nullptr;
    c.leaf_ops = L.use_tc && g->has_lstm && L.want_grad ? reinterpret_cast<uint4*>(ws + L.leaf_ops) : nullptr;
    c.all_leaves = reinterpret_cast<uint32_t*>(ws + L.all_leaves);
    c.loss_partial = reinterpret_cast<float*>(ws + L.loss_partial);
    c.repro = L.repro;
    c.dw_partial = L.repro ? reinterpret_cast<float*>(ws + L.dw_partial) : nullptr;
    c.dE_fix = L.repro ? reinterpret_cast<long long*>(ws + L.de_fix) : nullptr;
    c.head_fix = L.repro ? reinterpret_cast<long long*>(ws + L.head_fix) : nullptr;
    c.rank_tmp = L.repro ? reinterpret_cast<uint32_t*>(ws + L.rank_tmp) : nullptr;
    c.node_info = L.repro ? reinterpret_cast<uint2*>(ws + L.node_info) : nullptr;
    c.canon_hist = L.repro ? reinterpret_cast<uint32_t*>(ws + L.canon_hist) : nullptr;
    c.canon_cap = L.canon_cap;
    c.loss_out = out->loss;
    c.ctl = reinterpret_cast<Control*>(ws + L.ctl);
    c.wave_limit = L.wave_cap ? L.wave_cap : 1u << 24;
    if (S->wave_limit > 0) c.wave_limit = (uint32_t)std::min<long long>(S->wave_limit, c.wave_limit);
    c.probe_mode = S->probe_mode;
    c.spin_limit = S->wait_cycles > 0 ? S->wait_cycles : (long long)S->clock_khz * 2000ll;       // default: about two seconds of SM clock
}

int rdf_check_common(rdf_graph* g, const rdf_batch* in, const rdf_params* params, rdf_outputs* out, void* ws) {
    if (!g || !in || !out || !ws) return RDF_ERR_BAD_ARG;
    if ((uintptr_t)ws & 255) return RDF_ERR_BAD_ARG;
    if (g->uses_tree) {
        if (!in->tree_root || !in->left || !in->right || !in->tok || in->N <= 0) return RDF_ERR_BAD_ARG;
    } else if (!in->x) {
        return RDF_ERR_BAD_ARG;
    }
    if (g->has_vector_ops) {
        if (!params || !params->E || !params->W || !params->b || !out->h_root) return RDF_ERR_BAD_ARG;
        if (params->D != params->H) return RDF_ERR_UNSUPPORTED;
        if (g->has_lstm && (!params->W_x || !params->b_x)) return RDF_ERR_BAD_ARG;
        if (params->compute != RDF_F32 && params->compute != RDF_BF16) return RDF_ERR_BAD_ARG;
    } else if (!out->y) {
        return RDF_ERR_BAD_ARG;
    }
    if (out->trace && (!out->trace_count || out->trace_capacity <= 0)) return RDF_ERR_BAD_ARG;
    return RDF_OK;
}

// zero what must start at zero, upload the program, seed, run all waves
int rdf_launch_forward(rdf_graph* g, const rdf_batch* in, rdf_outputs* out, char* ws, const Layout& L, ExecState* S,
                       DevCtx& c, cudaStream_t stream) {
    rdf_mark(S, 0, stream);
    S->launches = 0;
    CUDA_OK(cudaMemsetAsync(ws + L.ctl, 0, 4096, stream));
    if (L.wave_cap) CUDA_OK(cudaMemsetAsync(ws + L.height_ends, 0, ((size_t)L.wave_cap + 2) * sizeof(uint32_t), stream));
    if (g->tag_mode == RDF_TAGS_FRAME) {
        bool wide = false;                        // an operator with more than two tagged inputs
        for (const MatchNode& m : g->match) wide = wide || m.n_ports > 2;
        if (L.pair_bytes) CUDA_OK(cudaMemsetAsync(ws + L.pair_slots, 0, L.pair_bytes, stream));
        if (wide && L.arrived_bytes) CUDA_OK(cudaMemsetAsync(ws + L.arrived, 0, L.arrived_bytes, stream));
    }
    if (L.table_bytes) CUDA_OK(cudaMemsetAsync(ws + L.table, 0xFF, L.table_bytes, stream));
    {
        // the four program tables sit next to each other in the workspace (code first, constants last): one copy
        const size_t bytes = L.consts + g->consts.size() * sizeof(int64_t) - L.code;
        if (S->tables_bytes != bytes) {
            // page-locked, so that the copy below is asynchronous to the host (made once per graph)
            if (S->tables) { if (S->tables_pinned) cudaFreeHost(S->tables); else free(S->tables); }
            S->tables = nullptr; S->tables_bytes = 0;
            if (S->may_allocate) {
                CUDA_OK(cudaHostAlloc(reinterpret_cast<void**>(&S->tables), bytes, cudaHostAllocDefault));
                S->tables_pinned = true;
            } else {
                S->tables = static_cast<char*>(malloc(bytes));
                if (!S->tables) return RDF_ERR_CUDA;
                S->tables_pinned = false;
            }
            S->tables_bytes = bytes;
            memset(S->tables, 0, bytes);
            memcpy(S->tables, g->code.data(), g->code.size() * sizeof(VmInstr));
            if (!g->match.empty()) memcpy(S->tables + (L.match - L.code), g->match.data(), g->match.size() * sizeof(MatchNode));
            if (!g->labels.empty()) memcpy(S->tables + (L.labels - L.code), g->labels.data(), g->labels.size() * sizeof(LabelInfo));
            if (!g->consts.empty()) memcpy(S->tables + (L.consts - L.code), g->consts.data(), g->consts.size() * sizeof(int64_t));
        }
        CUDA_OK(cudaMemcpyAsync(ws + L.code, S->tables, bytes, cudaMemcpyHostToDevice, stream));
    }
    RDF_KERNEL(S, rdf_seed_kernel<<<(unsigned)((in->B + 255) / 256), 256, 0, stream>>>(c));
    CUDA_OK(cudaGetLastError());
    if (c.use_tc) {
        if (c.lstm) {
            RDF_KERNEL(S, rdf_pack_lstm_kernel<<<256, 256, 0, stream>>>(c));
            RDF_KERNEL(S, rdf_pack_e_kernel<<<1024, 256, 0, stream>>>(c));
        } else {
            RDF_KERNEL(S, rdf_pack_w_kernel<<<64, 256, 0, stream>>>(c));
        }
        CUDA_OK(cudaGetLastError());
    }
    rdf_mark(S, 1, stream);
    void* args[] = {(void*)&c};
    if (g->interleaved)
        RDF_KERNEL(S, CUDA_OK(cudaLaunchCooperativeKernel((void*)rdf_interleaved_kernel, dim3(S->grid), dim3(1024), args,
                                            (size_t)interleaved_smem_bytes(c.H), stream)));
    else
        RDF_KERNEL(S, CUDA_OK(cudaLaunchCooperativeKernel((void*)rdf_scheduler_kernel, dim3(S->grid), dim3(1024), args,
                                            2 * LQ_CAP * sizeof(Token), stream)));
    rdf_mark(S, 2, stream);
    if (g->interleaved) {
        // the states were computed between the token waves: only the root rows are left to copy out
        rdf_mark(S, 3, stream);
        rdf_mark(S, 4, stream);
        RDF_KERNEL(S, rdf_gather_roots_kernel<<<(unsigned)in->B, 128, 0, stream>>>(c, out->h_root));
        CUDA_OK(cudaGetLastError());
    } else if (g->has_vector_ops) {
        void* oargs[] = {(void*)&c};
        DevCtx co = c;
        if (c.use_tc) {
            // the cells listed by call depth, with the operand row that every invocation's state goes to
            int rc = encode_row_tiles(&c.tmap_z128, c.z_bf, c.cells_cap, (uint64_t)2 * c.Hp, 128);
            if (rc == RDF_OK) rc = encode_row_tiles(&c.tmap_z64, c.z_bf, c.cells_cap, (uint64_t)2 * c.Hp, 64);
            if (rc == RDF_OK) rc = rdf_launch_lists(in, ws, L, S, c, stream);
            if (rc != RDF_OK) return rc;
            rdf_mark(S, 3, stream);
            RDF_KERNEL(S, CUDA_OK(cudaLaunchCooperativeKernel((void*)rdf_operator_kernel<true>, dim3(S->grid), dim3(TC_THREADS), oargs,
                                                (size_t)L.tc_smem_fwd, stream)));
        } else {
            // the cells grouped by height; the operator kernel reads the grouped list in place of the scheduler's
            RDF_KERNEL(S, rdf_height_count_kernel<<<2 * S->grid, 256, 0, stream>>>(c, 0));
            RDF_KERNEL(S, rdf_height_scan_kernel<<<1, 1024, 0, stream>>>(c, 0));
            RDF_KERNEL(S, rdf_height_scatter_kernel<<<2 * S->grid, 256, 0, stream>>>(c, 0));
            CUDA_OK(cudaGetLastError());
            rdf_mark(S, 3, stream);
            co.cell_items = c.cell_sorted;
            oargs[0] = (void*)&co;
            S->last_clusters = c.n_groups > 1 ? c.n_groups : 0;
            if (c.n_groups > 1) RDF_KERNEL(S, rdf_height_split_kernel<<<S->grid, 256, 0, stream>>>(c, 40u * (uint32_t)c.n_groups, 0));
            // the leaves and the wide heights with the whole grid ...
            if (c.lstm)
                RDF_KERNEL(S, CUDA_OK(cudaLaunchCooperativeKernel((void*)rdf_operator_kernel<false>, dim3(S->grid), dim3(256), oargs,
                                                    thin_resident_bytes(c.lstm, c.H), stream)));
            else
                RDF_KERNEL(S, CUDA_OK(cudaLaunchCooperativeKernel((void*)rdf_operator_kernel<false, true>, dim3(S->grid * S->rnn32_per_sm),
                                                    dim3(256), oargs, thin_resident_bytes(0, c.H), stream)));
            if (c.n_groups > 1) {
                // ... the narrow ones cluster by cluster of instances (the kernel leaves at once when the grouped table
                // did not fit and the grid-wide kernel did all the work)
                cudaLaunchConfig_t cfg = {};
                cudaLaunchAttribute at[1];
                at[0].id = cudaLaunchAttributeClusterDimension;
                at[0].val.clusterDim.x = CLUSTER_CTAS; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
                cfg.gridDim = dim3(c.n_groups * CLUSTER_CTAS); cfg.blockDim = dim3(256);
                cfg.dynamicSmemBytes = cluster_smem_bytes(c.H); cfg.stream = stream;
                cfg.attrs = at; cfg.numAttrs = 1;
                switch (cluster_cols_per_block(c.H)) {
                    case 8: RDF_KERNEL(S, CUDA_OK(cudaLaunchKernelEx(&cfg, rdf_operator_cluster_kernel<8>, co))); break;
                    case 16: RDF_KERNEL(S, CUDA_OK(cudaLaunchKernelEx(&cfg, rdf_operator_cluster_kernel<16>, co))); break;
                    case 32: RDF_KERNEL(S, CUDA_OK(cudaLaunchKernelEx(&cfg, rdf_operator_cluster_kernel<32>, co))); break;
                    default: RDF_KERNEL(S, CUDA_OK(cudaLaunchKernelEx(&cfg, rdf_operator_cluster_kernel<48>, co))); break;
                }
            }
        }
        rdf_mark(S, 4, stream);
        RDF_KERNEL(S, rdf_gather_roots_kernel<<<(unsigned)in->B, 128, 0, stream>>>(c, out->h_root));
        CUDA_OK(cudaGetLastError());
    } else {
        rdf_mark(S, 3, stream);
        rdf_mark(S, 4, stream);
    }
    if (out->trace)
        CUDA_OK(cudaMemcpyAsync(out->trace_count, &c.ctl->trace_count, sizeof(uint64_t), cudaMemcpyDeviceToDevice, stream));
    rdf_mark(S, 5, stream);
    S->last_ctl = c.ctl;
    S->last_stream = stream;
    S->ran = true;
    return RDF_OK;
}

int rdf_launch_lists(const rdf_batch* in, char* ws, const Layout& L, ExecState* S, DevCtx& c, cudaStream_t stream) {
    const int n_seg = (int)(in->max_invocations / LIST_SEG) + 1;
    uint2* seg = reinterpret_cast<uint2*>(ws + L.list_seg);
    RDF_KERNEL(S, rdf_list_count_kernel<<<n_seg, 256, 0, stream>>>(c, seg));
    RDF_KERNEL(S, rdf_list_scan_kernel<<<1, 1024, 0, stream>>>(c, seg, n_seg));
    RDF_KERNEL(S, rdf_list_fill_kernel<<<n_seg, 256, 0, stream>>>(c, seg));
    RDF_KERNEL(S, rdf_list_ends_kernel<<<2 * S->grid, 256, 0, stream>>>(c, seg));
    RDF_KERNEL(S, rdf_wave_compact_kernel<<<1, 1024, 0, stream>>>(c));
    if (c.repro) {                                  // the cells of every depth in argument order
        for (int leaves = c.lstm ? 1 : 0; leaves >= 0; --leaves) {     // (the leaves first: the cells' positions are used afterwards)
            // linear-time ranks over the node indices; the quadratic kernel takes over when they do not apply
            CUDA_OK(cudaMemsetAsync(c.node_info, 0, (size_t)std::max<long long>(in->N, 1) * sizeof(uint2), stream));
            CUDA_OK(cudaMemsetAsync(c.canon_hist, 0, ((size_t)c.canon_cap + 1) * sizeof(uint32_t), stream));
            const int seg_blocks = (int)std::min<long long>((in->N / CANON_SEG + 1 + 7) / 8, 8 * S->grid);
            RDF_KERNEL(S, rdf_canon_node_kernel<<<2 * S->grid, 256, 0, stream>>>(c, leaves));
            RDF_KERNEL(S, rdf_canon_sweep_kernel<<<seg_blocks, 256, 0, stream>>>(c, leaves, 0));
            RDF_KERNEL(S, rdf_canon_colscan_kernel<<<16, 256, 0, stream>>>(c));
            RDF_KERNEL(S, rdf_canon_sweep_kernel<<<seg_blocks, 256, 0, stream>>>(c, leaves, 1));
            RDF_KERNEL(S, rdf_canon_keys_kernel<<<2 * S->grid, 256, 0, stream>>>(c, leaves));
            RDF_KERNEL(S, rdf_canon_rank_kernel<<<4 * S->grid, 256, 0, stream>>>(c, leaves));
            RDF_KERNEL(S, rdf_canon_scatter_kernel<<<2 * S->grid, 256, 0, stream>>>(c, leaves));
        }
    }
    if (c.zdst) RDF_KERNEL(S, rdf_list_zdst_kernel<<<2 * S->grid, 256, 0, stream>>>(c));
    CUDA_OK(cudaGetLastError());
    return RDF_OK;
}

// The cells grouped again for the clustered gradient pass: by (cluster of their instance, call depth).  Reuses the
// grouped list and the bucket table of the forward pass, which is over.
int rdf_launch_depth_groups(char* ws, const Layout& L, ExecState* S, DevCtx& c, cudaStream_t stream) {
    if (c.n_groups <= 1) return RDF_OK;
    CUDA_OK(cudaMemsetAsync(ws + L.height_ends, 0, ((size_t)L.wave_cap + 2) * sizeof(uint32_t), stream));
    RDF_KERNEL(S, rdf_height_count_kernel<<<2 * S->grid, 256, 0, stream>>>(c, 1));
    RDF_KERNEL(S, rdf_height_scan_kernel<<<1, 1024, 0, stream>>>(c, 1));
    RDF_KERNEL(S, rdf_height_scatter_kernel<<<2 * S->grid, 256, 0, stream>>>(c, 1));
    RDF_KERNEL(S, rdf_height_split_kernel<<<S->grid, 256, 0, stream>>>(c, 40u * (uint32_t)c.n_groups, 1));
    CUDA_OK(cudaGetLastError());
    return RDF_OK;
}

void rdf_exec_release(rdf_graph* g) {
    ExecState* S = static_cast<ExecState*>(g->dev);
    if (S && S->have_events)
        for (cudaEvent_t e : S->ev) cudaEventDestroy(e);
    if (S && S->tables) { if (S->tables_pinned) cudaFreeHost(S->tables); else free(S->tables); }
    delete S;
    g->dev = nullptr;
}

extern "C" int rdf_workspace_bytes(const rdf_graph* g, const rdf_batch* in, const rdf_params* params, int want_grad,
                                   size_t* bytes) {
    if (!bytes) return RDF_ERR_BAD_ARG;
    Layout L;
    int rc = rdf_make_layout(g, in, params, want_grad, L);
    if (rc != RDF_OK) return rc;
    *bytes = L.total;
    return RDF_OK;
}

extern "C" int rdf_eval(rdf_graph* g, const rdf_batch* in, const rdf_params* params, rdf_outputs* out, void* workspace,
                        size_t workspace_bytes, void* stream) {
    int rc = rdf_check_common(g, in, params, out, workspace);
    if (rc != RDF_OK) return rc;
    Layout L;
    rc = rdf_make_layout(g, in, params, 0, L);
    if (rc != RDF_OK) return rc;
    if (workspace_bytes < L.total) return RDF_ERR_WORKSPACE_TOO_SMALL;
    ExecState* S = rdf_state_of(g);
    rc = rdf_prepare_device(g, S);
    if (rc != RDF_OK) return rc;
    DevCtx c;
    rdf_fill_ctx(g, in, params, out, static_cast<char*>(workspace), L, S, c);
    return rdf_launch_forward(g, in, out, static_cast<char*>(workspace), L, S, c, static_cast<cudaStream_t>(stream));
}

extern "C" int rdf_last_status(rdf_graph* g, rdf_stats* s) {
    if (!g || !s) return RDF_ERR_BAD_ARG;
    ExecState* S = rdf_state_of(g);
    memset(s, 0, sizeof(*s));
    if (!S->ran) return RDF_OK;
    if (cudaStreamSynchronize(S->last_stream) != cudaSuccess) return RDF_ERR_CUDA;
    Control h;
    if (cudaMemcpy(&h, S->last_ctl, sizeof(Control), cudaMemcpyDeviceToHost) != cudaSuccess) return RDF_ERR_CUDA;
    s->status = h.status;
    s->waves = h.waves; s->waves_backward = h.waves_backward; s->max_wave_tokens = h.max_wave_tokens;
    s->invocations = h.invocations; s->tokens = h.tokens;
    s->store_inserts = h.store_inserts; s->store_matches = h.store_matches; s->store_probes = h.store_probes;
    s->max_probe = h.max_probe; s->max_depth = h.max_depth; s->cells = h.cells; s->leaves = h.leaves;
    s->cycles_schedule = h.cyc[0]; s->cycles_batch = h.cyc[1]; s->cycles_barrier = h.cyc[2];
    s->cycles_bwd_frames = h.cyc[3]; s->cycles_bwd_batch = h.cyc[4]; s->cycles_bwd_barrier = h.cyc[5];
    s->kernel_launches = S->launches;
    s->clusters = (uint32_t)S->last_clusters;
    return h.status;
}

extern "C" int rdf_set_limits(rdf_graph* g, long long wait_cycles, long long wave_limit) {
    if (!g || wait_cycles < 0 || wave_limit < 0) return RDF_ERR_BAD_ARG;
    ExecState* S = rdf_state_of(g);
    S->wait_cycles = wait_cycles;
    S->wave_limit = wave_limit;
    return RDF_OK;
}

extern "C" int rdf_set_store(rdf_graph* g, int probe_mode, long long hash_slots) {
    if (!g || (probe_mode != RDF_PROBE_THREAD && probe_mode != RDF_PROBE_WARP) || hash_slots < 0) return RDF_ERR_BAD_ARG;
    ExecState* S = rdf_state_of(g);
    S->probe_mode = probe_mode;
    S->hash_slots = hash_slots;
    return RDF_OK;
}

extern "C" int rdf_set_profiling(rdf_graph* g, int enable) {
    if (!g) return RDF_ERR_BAD_ARG;
    ExecState* S = rdf_state_of(g);
    if (enable && !S->have_events) {
        for (cudaEvent_t& e : S->ev) CUDA_OK(cudaEventCreate(&e));
        S->have_events = true;
    }
    S->profiling = enable != 0;
    S->n_phases = 0;
    return RDF_OK;
}

extern "C" int rdf_last_phase_ms(rdf_graph* g, float* ms, int capacity, int* n) {
    if (!g || !ms || !n) return RDF_ERR_BAD_ARG;
    ExecState* S = rdf_state_of(g);
    *n = 0;
    if (!S->profiling || !S->have_events || S->n_phases == 0) return RDF_OK;
    CUDA_OK(cudaEventSynchronize(S->ev[S->n_phases]));
    for (int k = 0; k < S->n_phases && k < capacity; ++k) {
        CUDA_OK(cudaEventElapsedTime(&ms[k], S->ev[k], S->ev[k + 1]));
        *n = k + 1;
    }
    return RDF_OK;
}

// ===========================================================================
// fp32 FMA rate of the device (the denominator for the fp32 cell kernels)
// ===========================================================================
static __device__ float rdf_probe_sink;

__global__ void __launch_bounds__(256) rdf_probe_fma_kernel(int iters, float seed) {
    // eight independent chains per thread, operands in registers: nothing but the FMA pipe is busy
    float a0 = seed + threadIdx.x, a1 = a0 + 1.f, a2 = a0 + 2.f, a3 = a0 + 3.f, a4 = a0 + 4.f, a5 = a0 + 5.f, a6 = a0 + 6.f,
          a7 = a0 + 7.f;
    const float m = 0.999f, b = 1e-3f;
#pragma unroll 4
    for (int i = 0; i < iters; ++i) {
        a0 = fmaf(a0, m, b); a1 = fmaf(a1, m, b); a2 = fmaf(a2, m, b); a3 = fmaf(a3, m, b);
        a4 = fmaf(a4, m, b); a5 = fmaf(a5, m, b); a6 = fmaf(a6, m, b); a7 = fmaf(a7, m, b);
    }
    const float t = ((a0 + a1) + (a2 + a3)) + ((a4 + a5) + (a6 + a7));
    if (t == -1.2345e30f) rdf_probe_sink = t;          // never true: keeps the chains alive
}

extern "C" int rdf_probe_fp32_fma(double* tflops, void* stream_v) {
    if (!tflops) return RDF_ERR_BAD_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    int dev = 0, sms = 0;
    CUDA_OK(cudaGetDevice(&dev));
    CUDA_OK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    cudaEvent_t e0, e1;
    CUDA_OK(cudaEventCreate(&e0));
    CUDA_OK(cudaEventCreate(&e1));
    const int iters = 1 << 15, blocks = sms * 8;
    double best = 0.0;
    int rc = RDF_OK;
    for (int rep = 0; rep < 4 && rc == RDF_OK; ++rep) {                    // the first repetition warms up
        cudaEventRecord(e0, stream);
        rdf_probe_fma_kernel<<<blocks, 256, 0, stream>>>(iters, 1.f);
        cudaEventRecord(e1, stream);
        float ms = 0.f;
        if (cudaEventSynchronize(e1) != cudaSuccess || cudaEventElapsedTime(&ms, e0, e1) != cudaSuccess || ms <= 0.f) rc = RDF_ERR_CUDA;
        else if (rep > 0) best = std::max(best, 2.0 * 8.0 * iters * 256.0 * blocks / (ms * 1e-3) / 1e12);
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    *tflops = best;
    return rc;
}

// ===========================================================================
// Evaluation without any caller-supplied or freshly allocated scratch memory
// ===========================================================================
// Built-in scratch: lives in the library image, so every GPU that loads the
// library holds these 16 MiB until the process exits.
static __device__ __align__(256) unsigned char rdf_builtin_scratch[RDF_NOALLOC_SCRATCH_BYTES];

namespace {
// Device address of the array above, looked up once per device.  In host code
// the array's name is only a handle for the runtime; kernels need the address
// that cudaGetSymbolAddress returns for the device that is current.
const int kMaxDevices = 64;
void* g_builtin_scratch[kMaxDevices] = {};
std::mutex g_builtin_scratch_lock;      // first calls may come from several host threads

int builtin_scratch(void** out) {
    int dev = 0;
    CUDA_OK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return RDF_ERR_BAD_ARG;
    std::lock_guard<std::mutex> hold(g_builtin_scratch_lock);
    if (!g_builtin_scratch[dev]) {
        void* p = nullptr;
        CUDA_OK(cudaGetSymbolAddress(&p, rdf_builtin_scratch));
        if (!p) return RDF_ERR_CUDA;
        g_builtin_scratch[dev] = p;
    }
    *out = g_builtin_scratch[dev];
    return RDF_OK;
}
}  // namespace

extern "C" int rdf_eval_noalloc(rdf_graph* g, const rdf_batch* in, const rdf_params* params, rdf_outputs* out,
                                void* stream) {
    if (!g || !in || !out) return RDF_ERR_BAD_ARG;
    Layout L;
    int rc = rdf_make_layout(g, in, params, 0, L);
    if (rc != RDF_OK) return rc;
    if (L.total > (size_t)RDF_NOALLOC_SCRATCH_BYTES) return RDF_ERR_WORKSPACE_TOO_SMALL;   // batch too large for the built-in array
    void* ws = nullptr;
    rc = builtin_scratch(&ws);
    if (rc != RDF_OK) return rc;
    rc = rdf_check_common(g, in, params, out, ws);
    if (rc != RDF_OK) return rc;
    ExecState* S = rdf_state_of(g);
    rc = rdf_prepare_device(g, S);
    if (rc != RDF_OK) return rc;
    DevCtx c;
    rdf_fill_ctx(g, in, params, out, static_cast<char*>(ws), L, S, c);
    // rdf_launch_forward clears the control block, the arrival counters and the hash tables
    // on the stream before the first kernel, so nothing of the previous call is read.
    S->may_allocate = false;                       // (no allocating CUDA call on this path: the program tables stay pageable)
    rc = rdf_launch_forward(g, in, out, static_cast<char*>(ws), L, S, c, static_cast<cudaStream_t>(stream));
    S->may_allocate = true;
    return rc;
}
