// Device-side data structures and primitives of the executor: tokens, packed
// tags, frames, the token store (hash and dense forms), wave queues, the grid
// barrier.  Everything lives in the caller's workspace.
//
// Memory rule of the persistent kernels: data that one SM writes and another
// reads in a later phase is read through L2 (__ldcg / __ldcv), never through
// the non-coherent L1.
#pragma once
#include <cooperative_groups.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "rdf_internal.h"

namespace cg = cooperative_groups;

// A token <tag, datum> on its way to the segment that starts at `pc`.
struct __align__(16) Token {
    uint64_t tag;
    int64_t  datum;
    uint32_t pc;
    uint32_t aux;
    uint64_t pad;
};
static_assert(sizeof(Token) == 32, "two 128-bit words");

// Frame record (frame-form tags): the paper's frame with its label field and
// the reference to the previous scope (Section 5.1).
struct __align__(16) Frame {
    uint32_t parent;
    uint32_t label;               // [7:0] label i of the Call_i that made the frame, [31:8] the scheduler wave it fired in
    int64_t  arg;
};
static const uint32_t FRAME_LABEL_MASK = 0xFFu;
static const uint32_t CHILD_L_MARK = 0xFFFFFFFDu, CHILD_R_MARK = 0xFFFFFFFEu;   // CellItem.r of a unary vector operator (no frame has these ids)
static const int INTERLEAVED_MAX_H = 256;          // interleaved execution stages 2 H floats per warp in shared memory
static const uint32_t LOOP_LABEL = 0xFFu;     // label field of a loop frame (Enter), which no call site has
// A tag in frame form: the frame id in the low half; for a loop frame the iteration counter in the high half
// (Section 5.1: a tag is a pair of an iteration number and a pointer into the frame stack).
__device__ __forceinline__ uint32_t frame_of(uint64_t tag) { return (uint32_t)tag; }
static const int FRAME_WAVE_SHIFT = 8;

// Hash-store slot: a parked operand keyed by the packed tag.
struct __align__(16) Slot {
    uint64_t key;
    int64_t  val;
};
static const uint64_t SLOT_EMPTY = ~0ull;     // depth field 63: never a tag

struct __align__(16) CellItem {               // one ready cell: state of `out` from states of l, r
    uint32_t out, l, r;
    uint32_t height;                          // 1 + the larger height of its operands (leaves: 0)
};
struct __align__(8) LeafItem {
    uint32_t slot;
    int32_t  tok;
};

// A counter that many warps hit with atomics in the same wave, alone on its 128-byte line: atomics on
// different counters then do not queue up behind each other in one L2 slice, and the polling of a
// barrier word does not compete with them.
struct alignas(128) HotCounter {
    uint32_t v;
};

// Counters and control words, one 4 KB block at the start of the workspace.
struct Control {
    HotCounter qcount[3];         // tokens in the queue of wave w at [w % 3]
    HotCounter cell_count;        // ready cells queued so far, all waves (length of cell_items)
    HotCounter leaf_count;        // ready leaves queued so far (length of leaf_items)
    HotCounter frame_count;
    HotCounter bar;               // grid barrier arrivals of the scheduler kernel (monotone)
    HotCounter bar2;              // barrier counter of the backward kernel
    HotCounter bar_ops;           // barrier counter of the operator kernel
    int32_t  status;
    uint32_t waves, waves_backward, max_wave_tokens, max_probe, max_depth;
    uint32_t all_cells;           // backward: cells seen so far (length of the all-cells list)
    uint32_t all_leaves;          // backward: leaves seen so far
    uint32_t resume_wave;         // wave index at which the grid carries on after a stretch of narrow waves
    uint32_t max_height;          // largest height of a cell of this call (operator waves run height by height)
    uint32_t h_split;             // clustered fp32 path: heights up to here are wide and fired by the whole grid, the rest cluster by cluster
    uint32_t d_split;             // clustered gradient pass: call depths (scheduler wave + 1) up to here are wide and run by the whole grid
    uint32_t n_depth_waves;       // scheduler waves that made calls = call depths of the run (length of the compacted wave_marks)
    unsigned long long invocations, tokens, store_inserts, store_matches, store_probes, cells, leaves;
    unsigned long long trace_count;
    unsigned long long cyc[6];    // block 0: forward schedule / batch / barrier, backward frames / batch / barrier
    float    loss;
    int32_t  forward_status;      // status word at the end of the forward pass and the loss head
};
static_assert(sizeof(Control) <= 4096, "the control block is 4 KB");

// A tensor map as the driver encodes it (128 opaque bytes; the host fills it with cuTensorMapEncodeTiled).
struct alignas(64) TensorMap { unsigned long long opaque[16]; };

struct DevCtx {
    // lowered program (copied into the workspace at every call)
    const VmInstr*   code;
    const MatchNode* match;
    const LabelInfo* labels;
    const int64_t*   consts;
    int n_code, n_match, n_labels, n_consts;
    int label_bits, tag_mode, result_entry_pc, n_ports_total, K;   // K = call sites per body (children per frame)
    // batch
    long long B, N;
    const int64_t* x;
    const int32_t *tree_root, *left, *right, *tok, *label;
    // wave queues
    Token*   q[2];
    uint32_t qcap;
    // frames (frame-form tags)
    Frame*    frames;
    uint32_t* finst;              // [frame_cap] fp32 tree networks: the instance (tree) an invocation belongs to, handed down
                                  // from caller to callee; instances never exchange tokens, so the cells of different
                                  // instances can be fired by different groups of thread blocks without a grid barrier
    int       n_groups;           // thread-block clusters of the clustered operator kernel (0: not used)
    uint64_t* frame_ptag;         // [frame_cap] programs with loops: the full tag below a frame (its frame id and, when
                                  // that frame is a loop's, the iteration counter in the high half)
    int       has_loops;
    uint32_t  frame_cap;
    int64_t*  frame_args;         // [frame_cap * 2]: parameters 1 and 2 of invocations of multi-parameter functions
    // token store, dense form.  Two-input operators: one 16-byte slot per (frame, match node), operand
    // and arrival exchanged in one atomic.  More inputs: one cell per (frame, port) and an arrival
    // counter per (frame, match node).
    Slot*     pair_slots;
    int64_t*  port_val;
    uint32_t* arrived;
    // token store, hash form: one open-addressing table per match node
    Slot*     table;
    uint64_t  table_cap;          // slots per match node, power of two
    // batched operators
    CellItem* cell_items;         // every cell in the order it became ready (wave after wave); the operator kernel
                                  // gets the copy sorted by height here
    CellItem* cell_sorted;        // the cells grouped by height: the operands of a cell of height k have heights < k, so
                                  // all cells of one height fire together whatever wave the scheduler found them in
    uint32_t* height_ends;        // [wave_cap + 2]: cells per height, then (after the scatter) the end of each group
    LeafItem* leaf_items;         // every leaf in the order it was reached
    uint32_t  work_cap;
    uint32_t* op_l;               // per frame: operand frames of the operator that made its state
    uint32_t* op_r;               //            (leaf: op_l = LEAF_MARK, op_r = token id)
    float*    arena;              // [frame_cap, S] fp32 states: S = H (TreeRNN h) or 2H (TreeLSTM h then c)
    float*    gates;              // TreeLSTM under rdf_grad: [frame_cap, G] activated gates, later their gradients
    int       S, G, lstm;
    // tensor-core path (bf16 operands): bf16 copy of the states with row stride Hp, packed weights
    __nv_bfloat16* arena_bf;
    __nv_bfloat16* Wp;            // [Hp, 2Hp]   forward operand
    __nv_bfloat16* WTp;           // [2Hp, Hp]   gradient operand
    __nv_bfloat16* dz_bf;         // [frame_cap, Hp] bf16 dz rows of the cells (rdf_grad), row = position of the cell in
                                  // all_cells: the cells of a gradient wave are consecutive rows, read as plain 2D tiles
    uint32_t* cell_pos;           // per frame: position of a cell in all_cells (written with the lists; leaves: undefined)
    TensorMap tmap_dz128, tmap_dz64;   // dz_bf as [rows, Hp], 128-byte swizzle, boxes of 128 / 64 rows by 64 columns
    __nv_bfloat16* z_bf;          // [cells_cap, 2Hp] operand rows [h_l ; h_r] of the cells, row = position of the cell in
                                  // all_cells: every invocation writes its state into the half of its caller's row
                                  // that it feeds, so a tile of consecutive cells reads its operands as plain 2D tiles
    uint32_t* zdst;               // per frame: 2 * (position of the calling cell) + operand port, or NO_ZDST
    uint32_t  cells_cap;          // rows of z_bf / dz_bf that exist
    TensorMap tmap_z128, tmap_z64;     // z_bf as [rows, 2Hp]
    // TreeLSTM on tensor cores: Wp / WTp hold the slice-major W5p [5Hp, 2Hp] and WT5p [2Hp, 5Hp]
    __nv_bfloat16* Wxp;           // [3Hp, Hp] leaf projection, slice-major
    __nv_bfloat16* WxTp;          // [Hp, 3Hp] its transpose (operand of the embedding gradient)
    __nv_bfloat16* E_bf;          // [V, Hp] embedding table in bf16
    __nv_bfloat16* dg_bf;         // [frame_cap, 5Hp] bf16 gate gradients (rdf_grad)
    int       Hp, use_tc;
    // parameters
    int H, D, V, n_classes, compute;
    const float *E, *W, *b, *W_x, *b_x, *W_s, *b_s;
    // outputs
    int64_t* y;                   // integer results / for vector programs the frame holding the root state
    rdf_trace_rec* trace;
    long long trace_cap;
    // gradient pass
    float*    dhp;                // [frame_cap, S]: gradient arriving from the caller (dh, and dc for the TreeLSTM);
                                  //                 TreeRNN: overwritten by dz (cell) / dh (leaf)
    float*    dlog;               // [frame_cap, 8]: softmax - onehot per invocation
    uint4*    wave_marks;         // [wave_cap], filled by the list kernels: entry k = {first frame, one past the last frame,
                                  // first cell, one past the last cell (positions in all_cells)} of the k-th scheduler
                                  // wave that made calls.  Frame ids are handed out in wave order, so the invocations
                                  // of one call depth are one id range -- one wave of the gradient pass, and (from
                                  // the deepest one up) one wave of the tensor-core operator kernel
    uint32_t  wave_cap;
    uint32_t* all_cells;          // every cell frame, in backward wave order
    uint4*    cell_ops;           // {cell frame, left operand frame, right operand frame, 1} in all_cells order
    uint4*    leaf_ops;           // {leaf frame, token id, 0, 1} in all_leaves order
    uint32_t* all_leaves;         // every leaf frame
    float*    loss_partial;       // per-block partial sums of the loss
    // reproducible mode (tensor-core path): sums that do not depend on the order in which thread blocks get to them
    int       repro;
    float*    dw_partial;         // split-K partial tiles of the weight gradient [block, 256, 256] (also the per-block rows
                                  // of the column sums), added up in block order
    long long* dE_fix;            // [V, D] the embedding gradient in 64-bit fixed point (integer sums are exact)
    long long* head_fix;          // [n_classes * (H + 1) + 1] dW_s, db_s and the loss in fixed point
    uint2*    node_info;          // [N] reproducible mode: per tree node {list position + 1, depth + 1} of the cell (leaf) it carries
    uint32_t* canon_hist;         // [canon_cap + 1] entries per (segment of nodes, depth); the last word flags the fallback
    uint32_t  canon_cap;
    uint32_t* rank_tmp;           // [frame_cap] scratch of the pass that puts the cells of a depth in argument order
    float    *dE, *dW, *db, *dW_x, *db_x, *dW_s, *db_s;
    float*    loss_out;
    // control
    Control*  ctl;
    uint32_t  wave_limit;
    int       probe_mode;         // hash store: 0 = every thread probes for itself, 1 = the threads of a warp probe together
    long long spin_limit;         // clock64 ticks a barrier wait may last
};

static const uint32_t LEAF_MARK = 0xFFFFFFFFu;

// How many groups the ready cells are sorted into (by instance, then by height): the clusters of the clustered
// operator kernel when the (group, height) table fits the space of the height table, else one group (all cells
// by height, fired by the whole grid).  Every kernel of a call computes the same answer from the same words.
// Shallow batches stay with the grid-wide kernel: a few dozen waves are too few for the second kernel to pay.
static const uint32_t CLUSTER_MIN_HEIGHT = 64;
__device__ __forceinline__ uint32_t cell_groups(const DevCtx& c) {
    const uint64_t stride = (uint64_t)min(c.ctl->max_height, c.wave_cap) + 1u;
    return c.n_groups > 1 && stride > CLUSTER_MIN_HEIGHT && (uint64_t)c.n_groups * stride <= (uint64_t)c.wave_cap + 2u
               ? (uint32_t)c.n_groups : 1u;
}
// The same for the gradient pass, whose waves go by call depth (the scheduler wave that created the frame): cells grouped
// by (cluster of their instance, scheduler wave + 1).
__device__ __forceinline__ uint32_t depth_groups(const DevCtx& c) {
    const uint64_t stride = (uint64_t)min(c.ctl->waves, c.wave_cap) + 1u;
    return cell_groups(c) > 1u && (uint64_t)c.n_groups * stride <= (uint64_t)c.wave_cap + 2u ? (uint32_t)c.n_groups : 1u;
}
__device__ __forceinline__ uint32_t bucket_groups(const DevCtx& c, int by_depth) { return by_depth ? depth_groups(c) : cell_groups(c); }
__device__ __forceinline__ uint32_t bucket_stride(const DevCtx& c, int by_depth) {
    return min(by_depth ? c.ctl->waves : c.ctl->max_height, c.wave_cap) + 1u;
}
static const uint32_t NO_ZDST = 0xFFFFFFFFu;

// thread-block clusters of the clustered fp32 kernels (forward cells, gradient waves)
static const int CLUSTER_CTAS = 8;
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// 64-bit fixed point, 2^-36 per unit (|sum| < 1.3e8, resolution 1.5e-11): integer additions commute exactly
#define RDF_FIX_SCALE 68719476736.0f
__device__ __forceinline__ long long to_fix(float v) { return __float2ll_rn(v * RDF_FIX_SCALE); }
__device__ __forceinline__ void fix_add(long long* p, long long v) {
    atomicAdd(reinterpret_cast<unsigned long long*>(p), (unsigned long long)v);
}
__device__ __forceinline__ float from_fix(long long v) { return (float)((double)v * (1.0 / (double)RDF_FIX_SCALE)); }

// ---------------------------------------------------------------- utilities
__device__ __forceinline__ void set_status(const DevCtx& c, int code) { atomicCAS(&c.ctl->status, 0, code); }

__device__ __forceinline__ uint32_t ld_volatile_u32(const uint32_t* p) {
    return *reinterpret_cast<const volatile uint32_t*>(p);
}
__device__ __forceinline__ int32_t ld_volatile_i32(const int32_t* p) {
    return *reinterpret_cast<const volatile int32_t*>(p);
}

// One atomic per converged group of threads instead of one per thread.
__device__ __forceinline__ uint32_t aggregated_inc(uint32_t* counter) {
    cg::coalesced_group g = cg::coalesced_threads();
    uint32_t base = 0;
    if (g.thread_rank() == 0) base = atomicAdd(counter, g.size());
    return g.shfl(base, 0) + g.thread_rank();
}

// Two counters bumped by the same converged group: both atomics are in flight together (one L2 round trip
// instead of two on the token's critical path).
__device__ __forceinline__ void aggregated_inc2(uint32_t* ca, uint32_t* cb, uint32_t& a, uint32_t& b) {
    cg::coalesced_group g = cg::coalesced_threads();
    uint32_t ba = 0, bb = 0;
    if (g.thread_rank() == 0) {
        ba = atomicAdd(ca, g.size());
        bb = atomicAdd(cb, g.size());
    }
    a = g.shfl(ba, 0) + g.thread_rank();
    b = g.shfl(bb, 0) + g.thread_rank();
}

// The same for n consecutive places on each counter per thread (a pair of calls): the thread's places are a .. a + n - 1.
__device__ __forceinline__ void aggregated_inc2n(uint32_t* ca, uint32_t* cb, uint32_t n, uint32_t& a, uint32_t& b) {
    cg::coalesced_group g = cg::coalesced_threads();
    uint32_t ba = 0, bb = 0;
    if (g.thread_rank() == 0) {
        ba = ca ? atomicAdd(ca, n * g.size()) : 0u;
        bb = atomicAdd(cb, n * g.size());
    }
    a = g.shfl(ba, 0) + n * g.thread_rank();
    b = g.shfl(bb, 0) + n * g.thread_rank();
}

// Grid-wide barrier with a bounded wait.  All blocks of the (cooperatively
// launched, hence co-resident) grid call it the same number of times.  The
// counter only grows; generation k is complete when it reaches k * gridDim.x.
// Returns false when the wait expired or any block reported an error; the
// caller then leaves the kernel.
// The arrival is a release reduction (no value comes back, so the thread goes straight on to poll) and the
// wait polls with acquire loads (GPU scope): what a block wrote before the barrier is visible to every block
// that sees the full count, and no separate fence has to wait for the stores and atomics still in flight.
// The status word is looked at every few polls, so that a block that is still waiting when another block has
// reported an error leaves at once instead of waiting for its own limit.
__device__ __forceinline__ bool grid_barrier(const DevCtx& c, uint32_t* counter, uint32_t& generation) {
    __shared__ int ok;
    __syncthreads();
    if (threadIdx.x == 0) {
        ++generation;
        const uint32_t target = generation * gridDim.x;
        asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(counter) : "memory");
        const long long t0 = clock64();
        int good = 1;
        for (uint32_t polls = 0;; ++polls) {
            uint32_t seen;
            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(counter) : "memory");
            if (seen >= target) break;
            if (clock64() - t0 > c.spin_limit) {
                set_status(c, RDF_ERR_TIMEOUT);
                good = 0;
                break;
            }
            if ((polls & 15u) == 15u && ld_volatile_i32(&c.ctl->status) != 0) {
                good = 0;
                break;
            }
        }
        if (ld_volatile_i32(&c.ctl->status) != 0) good = 0;
        ok = good;
    }
    __syncthreads();
    return ok != 0;
}

// ------------------------------------------------------------------- queues
__device__ __forceinline__ void store_token(Token* dst_tok, uint64_t tag, int64_t datum, uint32_t pc) {
    uint4* dst = reinterpret_cast<uint4*>(dst_tok);
    dst[0] = make_uint4((uint32_t)tag, (uint32_t)(tag >> 32), (uint32_t)datum, (uint32_t)((uint64_t)datum >> 32));
    dst[1] = make_uint4(pc, 0u, 0u, 0u);
}

// The queue of a stretch of narrow waves that one block runs alone: the next wave's tokens stay in that
// block's shared memory (same slot numbering as the global queue; a token beyond the local capacity goes
// to its slot of the global queue, and the stretch ends there).
static const uint32_t LQ_CAP = 1024;
struct LocalQ {
    Token*    buf[2];        // shared memory, by wave parity
    uint32_t* count;         // shared memory, [3], by wave % 3
    uint32_t* ctr;           // shared memory, [3]: the frame, cell and leaf counters while one block runs a stretch of narrow
                             // waves alone (copied from the control block at its start, written back at its end): the
                             // reservations of a token cost a shared-memory atomic instead of an L2 round trip
};
enum { LQ_FRAMES = 0, LQ_CELLS = 1, LQ_LEAVES = 2 };

__device__ __forceinline__ void push_token(const DevCtx& c, const LocalQ* lq, uint32_t wave, uint64_t tag, int64_t datum,
                                           uint32_t pc) {
    if (lq) {
        const uint32_t idx = aggregated_inc(&lq->count[(wave + 1) % 3]);
        if (idx < LQ_CAP) store_token(&lq->buf[(wave + 1) & 1][idx], tag, datum, pc);
        else if (idx < c.qcap) store_token(&c.q[(wave + 1) & 1][idx], tag, datum, pc);
        else set_status(c, RDF_ERR_QUEUE_FULL);
        return;
    }
    const uint32_t idx = aggregated_inc(&c.ctl->qcount[(wave + 1) % 3].v);
    if (idx >= c.qcap) {
        set_status(c, RDF_ERR_QUEUE_FULL);
        return;
    }
    store_token(&c.q[(wave + 1) & 1][idx], tag, datum, pc);
}

__device__ __forceinline__ Token load_local_token(const Token* p) {       // from shared memory
    const uint4* src = reinterpret_cast<const uint4*>(p);
    const uint4 a = src[0], b = src[1];
    Token t;
    t.tag = (uint64_t)a.x | ((uint64_t)a.y << 32);
    t.datum = (int64_t)((uint64_t)a.z | ((uint64_t)a.w << 32));
    t.pc = b.x;
    t.aux = 0;
    t.pad = 0;
    return t;
}

// two coalesced 128-bit loads per token, through L2
__device__ __forceinline__ Token load_token(const Token* p) {
    const uint4* src = reinterpret_cast<const uint4*>(p);
    const uint4 a = __ldcg(src), b = __ldcg(src + 1);
    Token t;
    t.tag = (uint64_t)a.x | ((uint64_t)a.y << 32);
    t.datum = (int64_t)((uint64_t)a.z | ((uint64_t)a.w << 32));
    t.pc = b.x;
    t.aux = 0;
    t.pad = 0;
    return t;
}

// --------------------------------------------------------------------- tags
// Packed path form: [63:44] instance | [43:38] depth | [37:0] labels, innermost lowest.
__device__ __forceinline__ uint64_t path_root(long long instance) { return (uint64_t)instance << RDF_INST_SHIFT; }

// (parent: the tag below -- frame form: frame id and, in the high half, the iteration counter of a loop frame)
__device__ __forceinline__ void trace_rec(const DevCtx& c, uint64_t tag, int64_t value, uint32_t kind, uint32_t label,
                                          uint64_t parent) {
    if (!c.trace) return;
    const unsigned long long i = atomicAdd(&c.ctl->trace_count, 1ull);
    if ((long long)i < c.trace_cap) {
        rdf_trace_rec r;
        r.tag = tag; r.value = value; r.kind = kind; r.label = label;
        r.parent = c.tag_mode == RDF_TAGS_PATH ? 0u : (uint32_t)parent;
        r.instance = c.tag_mode == RDF_TAGS_PATH ? (uint32_t)(tag >> RDF_INST_SHIFT) : (uint32_t)(parent >> 32);
        c.trace[i] = r;
    }
}

// The record of a new frame (frame-form tags): its caller's frame, the label of the call site, the argument.
// The record also keeps the scheduler wave in which the call fired: ids are handed out wave after wave, so
// the frames of one wave are one id range, and the gradient pass finds the ranges from these fields.
__device__ __forceinline__ void frame_init(const DevCtx& c, const LabelInfo* labels, uint64_t tag, uint32_t label, int64_t arg,
                                           uint32_t id, uint32_t wave) {
    Frame f;
    f.parent = frame_of(tag); f.label = label | (wave << FRAME_WAVE_SHIFT); f.arg = arg;
    c.frames[id] = f;
    if (c.frame_ptag) c.frame_ptag[id] = tag;
    if (c.finst) c.finst[id] = __ldcg(&c.finst[frame_of(tag)]);
    trace_rec(c, id, arg, 0, label, tag);
}

// Call_i: <t, d> -> <i:t, d>.  Returns false (status set) when the tag cannot be formed.
__device__ __forceinline__ bool tag_push(const DevCtx& c, const LabelInfo* labels, uint64_t tag, uint32_t label,
                                         int64_t arg, uint64_t& out, uint32_t wave, const LocalQ* lq = nullptr) {
    if (c.tag_mode == RDF_TAGS_PATH) {
        const uint32_t depth = (uint32_t)(tag >> RDF_DEPTH_SHIFT) & 63u;
        if ((depth + 1) * (uint32_t)c.label_bits > (uint32_t)RDF_PATH_BITS) {
            set_status(c, RDF_ERR_TAG_OVERFLOW);
            return false;
        }
        const uint64_t path = tag & ((1ull << RDF_PATH_BITS) - 1);
        out = (tag & ~((1ull << RDF_INST_SHIFT) - 1)) | ((uint64_t)(depth + 1) << RDF_DEPTH_SHIFT) |
              ((path << c.label_bits) | label);
        trace_rec(c, out, arg, 0, label, 0);
        return true;
    }
    const uint32_t id = aggregated_inc(lq ? &lq->ctr[LQ_FRAMES] : &c.ctl->frame_count.v);
    if (id >= c.frame_cap) {
        set_status(c, RDF_ERR_FRAMES_FULL);
        return false;
    }
    frame_init(c, labels, tag, label, arg, id, wave);
    out = id;
    return true;
}

// Return_i: <i:t, d> -> <t, d>; yields the label i that the frame/tag carries.
__device__ __forceinline__ void tag_pop(const DevCtx& c, uint64_t tag, uint32_t& label, uint64_t& parent) {
    if (c.tag_mode == RDF_TAGS_PATH) {
        const uint32_t depth = (uint32_t)(tag >> RDF_DEPTH_SHIFT) & 63u;
        const uint64_t path = tag & ((1ull << RDF_PATH_BITS) - 1);
        label = (uint32_t)(path & ((1ull << c.label_bits) - 1));
        parent = (tag & ~((1ull << RDF_INST_SHIFT) - 1)) | ((uint64_t)(depth - 1) << RDF_DEPTH_SHIFT) |
                 (path >> c.label_bits);
    } else {
        const uint4 f = __ldcg(reinterpret_cast<const uint4*>(&c.frames[frame_of(tag)]));   // {parent, label, arg}
        label = f.y & FRAME_LABEL_MASK;
        parent = c.frame_ptag ? __ldcg(reinterpret_cast<const unsigned long long*>(&c.frame_ptag[frame_of(tag)])) : (uint64_t)f.x;
    }
}

// -------------------------------------------------------------- token store
__device__ __forceinline__ void cas128(Slot* addr, uint64_t cmp_lo, uint64_t cmp_hi, uint64_t new_lo,
                                       uint64_t new_hi, uint64_t& old_lo, uint64_t& old_hi) {
    asm volatile(
        "{\n"
        " .reg .b128 c, n, o;\n"
        " mov.b128 c, {%2, %3};\n"
        " mov.b128 n, {%4, %5};\n"
        " atom.global.cas.b128 o, [%6], c, n;\n"
        " mov.b128 {%0, %1}, o;\n"
        "}\n"
        : "=l"(old_lo), "=l"(old_hi)
        : "l"(cmp_lo), "l"(cmp_hi), "l"(new_lo), "l"(new_hi), "l"(addr)
        : "memory");
}

__device__ __forceinline__ uint64_t mix64(uint64_t k) {
    k ^= k >> 33; k *= 0xff51afd7ed558ccdull;
    k ^= k >> 33; k *= 0xc4ceb9fe1a85ec53ull;
    k ^= k >> 33;
    return k;
}

struct StoreCounters {
    uint32_t inserts = 0, matches = 0, probes = 0, max_probe = 0;
};

// Hash form, two-input operators: the first operand to arrive is parked under
// its tag, the second finds it and takes it (insert-or-consume).  A key is
// looked up exactly twice in the whole run, so a consumed entry is simply left
// in place; capacity is sized for all insertions of the run.
// Returns 1 and the partner's value when the match completed, 0 when parked,
// -1 when the table is full.
__device__ __forceinline__ int hash_insert_or_consume_from(const DevCtx& c, int node, uint64_t key, int64_t val,
                                                           int64_t& partner, StoreCounters& sc, uint64_t h) {
    Slot* tab = c.table + (size_t)node * c.table_cap;
    const uint64_t mask = c.table_cap - 1;
    for (uint64_t probe = 0; probe < c.table_cap; ++probe) {
        ++sc.probes;
        const uint4 raw = __ldcv(reinterpret_cast<const uint4*>(&tab[h]));
        uint64_t k = (uint64_t)raw.x | ((uint64_t)raw.y << 32);
        if (k == SLOT_EMPTY) {
            uint64_t old_lo, old_hi;
            cas128(&tab[h], SLOT_EMPTY, ~0ull, key, (uint64_t)val, old_lo, old_hi);
            if (old_lo == SLOT_EMPTY) {
                ++sc.inserts;
                if ((uint32_t)probe > sc.max_probe) sc.max_probe = (uint32_t)probe;
                return 0;
            }
            if (old_lo == key) {             // the partner took this slot meanwhile
                partner = (int64_t)old_hi;   // (the CAS returned key and value as one unit)
                ++sc.matches;
                return 1;
            }
        } else if (k == key) {
            // read key and value as one 128-bit unit: a failing CAS returns the slot's contents
            uint64_t old_lo, old_hi;
            cas128(&tab[h], SLOT_EMPTY, ~0ull, SLOT_EMPTY, ~0ull, old_lo, old_hi);
            partner = (int64_t)old_hi;
            ++sc.matches;
            return 1;
        }
        h = (h + 1) & mask;
    }
    return -1;
}
__device__ __forceinline__ int hash_insert_or_consume(const DevCtx& c, int node, uint64_t key, int64_t val,
                                                      int64_t& partner, StoreCounters& sc) {
    return hash_insert_or_consume_from(c, node, key, val, partner, sc, mix64(key) & (c.table_cap - 1));
}

// The same with cooperative probing: the threads of a warp that reach the store together look for one key at a
// time -- each inspects one of as many consecutive slots as there are threads (one coalesced load of 16 bytes per
// thread, 512 bytes for a full warp) and a ballot picks the first slot that holds the key or is empty.  When every
// key of the group has its slot, each thread finishes its own access there (128-bit CAS; should the slot have
// changed meanwhile it carries on alone from that slot).  Long probe sequences (a table filled close to capacity)
// cost one step per 32 slots instead of one per slot; at low load factors the per-thread form above needs about one
// load anyway and the rounds only add latency.
__device__ __forceinline__ int hash_insert_or_consume_group(const DevCtx& c, int node, uint64_t key, int64_t val,
                                                            int64_t& partner, StoreCounters& sc) {
    cg::coalesced_group g = cg::coalesced_threads();
    const uint32_t n = g.size(), me = g.thread_rank();
    const uint64_t mask = c.table_cap - 1;
    const uint64_t h = mix64(key) & mask;
    long long found = -1;
    for (uint32_t r = 0; r < n; ++r) {
        const uint64_t key_r = g.shfl(key, r), h_r = g.shfl(h, r);
        const Slot* tab_r = c.table + (size_t)g.shfl(node, r) * c.table_cap;
        for (uint64_t step = 0; step < c.table_cap; step += n) {
            const uint64_t idx = (h_r + step + me) & mask;
            const uint4 raw = __ldcv(reinterpret_cast<const uint4*>(&tab_r[idx]));
            const uint64_t k = (uint64_t)raw.x | ((uint64_t)raw.y << 32);
            const unsigned hits = g.ballot(k == key_r || k == SLOT_EMPTY);
            if (me == r) ++sc.probes;
            if (hits) {
                if (me == r) found = (long long)((h_r + step + (uint64_t)(__ffs(hits) - 1)) & mask);
                break;
            }
        }
    }
    if (found < 0) return -1;
    return hash_insert_or_consume_from(c, node, key, val, partner, sc, (uint64_t)found);
}

__device__ __forceinline__ void exch128(Slot* addr, uint64_t new_lo, uint64_t new_hi, uint64_t& old_lo, uint64_t& old_hi) {
    asm volatile(
        "{\n"
        " .reg .b128 n, o;\n"
        " mov.b128 n, {%2, %3};\n"
        " atom.global.exch.b128 o, [%4], n;\n"
        " mov.b128 {%0, %1}, o;\n"
        "}\n"
        : "=l"(old_lo), "=l"(old_hi)
        : "l"(new_lo), "l"(new_hi), "l"(addr)
        : "memory");
}

// Dense form (frame tags).  Two-input operator: the operand and the fact of its arrival go into the
// (frame, node) slot with one 128-bit exchange -- {1 + port, value}; the slot starts as {0, 0}.  The
// first operand finds the slot empty and stays there, the second gets the first one back.
// More inputs: the operand goes to its (frame, port) cell; the arrival that completes the set reads
// the others.  Returns 1 when complete.
// In a program with loops a slot serves every iteration of its loop frame (the iterations of one loop follow one
// another: Next fires when the whole body is done), so a completed match leaves the slot empty again.
__device__ __forceinline__ int dense_deliver(const DevCtx& c, const MatchNode& M, int node, uint64_t tag, int port,
                                             int64_t val, int64_t* regs, StoreCounters& sc) {
    const uint32_t frame = frame_of(tag);
    if (M.n_ports == 2) {
        uint64_t old_state, old_val;
        Slot* slot = &c.pair_slots[(size_t)frame * c.n_match + node];
        exch128(slot, 1ull + (uint64_t)port, (uint64_t)val, old_state, old_val);
        if (old_state == 0) {
            ++sc.inserts;
            return 0;
        }
        regs[port] = val;
        regs[1 - port] = (int64_t)old_val;
        if (c.has_loops) *reinterpret_cast<uint4*>(slot) = make_uint4(0u, 0u, 0u, 0u);
        ++sc.matches;
        return 1;
    }
    int64_t* cells = c.port_val + (size_t)frame * c.n_ports_total + M.port_base;
    cells[port] = val;
    __threadfence();
    const uint32_t before = atomicAdd(&c.arrived[(size_t)frame * c.n_match + node], 1u);
    if (before + 1 < (uint32_t)M.n_ports) {
        ++sc.inserts;
        return 0;
    }
    __threadfence();
    for (int p = 0; p < M.n_ports; ++p) regs[p] = __ldcv(reinterpret_cast<const long long*>(&cells[p]));
    if (c.has_loops) c.arrived[(size_t)frame * c.n_match + node] = 0u;
    ++sc.matches;
    return 1;
}
