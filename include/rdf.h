/* rdf.h -- recursive dataflow on one GPU: C boundary of the library.
 *
 * The library executes recursive function definitions as ONE static dataflow
 * graph extended with two tag operations (paper, Section 3):
 *
 *     Call_i   <t, d>   = <i:t, d>      tag-push on a recursive invocation
 *     Return_i <i:t, d> = <t, d>        tag-pop on return
 *
 * Tokens <tag, datum> of many concurrent invocations flow through the fixed
 * graph; an operator fires when all its inputs hold tokens with exactly the
 * same tag (Section 2.2), and all operators that are ready at the same time
 * fire as one batch on the device.
 *
 * Conventions for every function below
 *   - returns an int status: RDF_OK (0) or a negative RDF_ERR_* code; nothing
 *     throws, aborts or traps.  Conditions found on the device (capacity, tag
 *     overflow, an expired bounded wait) are written to a status word, all
 *     thread blocks leave, and the code is reported by rdf_last_status().
 *   - "host" pointers are ordinary CPU memory; "device" pointers are CUDA
 *     global memory of the current device, at least 16-byte aligned, owned by
 *     the caller and valid until the stream has passed the call.
 *   - rdf_eval / rdf_grad are stream-ordered: they enqueue work on `stream`
 *     (a cudaStream_t passed as void*) and return without synchronising.
 *     They allocate no device memory; all scratch comes from `workspace`.
 */
#ifndef RDF_H
#define RDF_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ------------------------------------------------------------------ status */
enum {
    RDF_OK = 0,
    RDF_ERR_BAD_PROGRAM = -1,        /* unknown callee, arity mismatch, no `result`, malformed expression */
    RDF_ERR_BAD_ARG = -2,            /* NULL or inconsistent argument */
    RDF_ERR_WORKSPACE_TOO_SMALL = -3,
    RDF_ERR_TAG_OVERFLOW = -4,       /* call depth x label bits exceeds the packed path field */
    RDF_ERR_STORE_FULL = -5,         /* token store has no free slot */
    RDF_ERR_FRAMES_FULL = -6,        /* more invocations than rdf_batch.max_invocations */
    RDF_ERR_QUEUE_FULL = -7,         /* more tokens in one wave than the queues hold */
    RDF_ERR_WAVE_LIMIT = -8,         /* guard against recursion that never reaches a base case */
    RDF_ERR_TIMEOUT = -9,            /* a bounded device-side wait expired */
    RDF_ERR_CUDA = -10,              /* a CUDA runtime call failed */
    RDF_ERR_UNSUPPORTED = -11        /* valid program outside what the device executor lowers */
};

/* ----------------------------------------------------------------- program
 * A program is a set of function definitions, one of which is `result`
 * (Section 3, the statement of the transformation's input).  Each definition
 * is an expression DAG over its formal parameters.  A CALL node is one of the
 * function-call nodes of Section 2.4, Figure 2; IF is the Switch/Merge
 * conditional of the same figure.
 */
typedef enum {
    RDF_OP_PARAM = 0,    /* imm = parameter index                                   */
    RDF_OP_CONST,        /* imm = value                                             */
    RDF_OP_ADD, RDF_OP_SUB, RDF_OP_MUL, RDF_OP_MAX,   /* a, b                       */
    RDF_OP_LT, RDF_OP_EQ,                             /* a, b -> 0/1                */
    RDF_OP_IF,           /* a = condition, b = then, c = else; the condition may contain calls (the Switch then fires
                            when they have returned; needs RDF_TAGS_FRAME when a branch reads a parameter) */
    RDF_OP_CALL,         /* imm = callee function index; a, b, c = one argument expression per formal
                            parameter of the callee (up to three); an argument may itself be a call */
    /* accessors on the batch's flat tree arrays; operand = node index           */
    RDF_OP_IS_LEAF, RDF_OP_LEFT, RDF_OP_RIGHT, RDF_OP_TOK,
    /* vector-valued operators of the tree networks                               */
    RDF_OP_EMBED,        /* a = token id          -> E[tok]                         */
    RDF_OP_CELL_RNN,     /* a, b = child states   -> tanh(W [a; b] + b)             */
    RDF_OP_LEAF_LSTM,    /* a = token id          -> (h, c) of a TreeLSTM leaf      */
    RDF_OP_CELL_LSTM,    /* a, b = child states   -> (h, c) of a binary TreeLSTM    */
    RDF_OP_NODE_LOSS,    /* a = state, b = node index; passes the state through and
                            marks the invocation as a term of the summed per-node
                            softmax cross-entropy loss that rdf_grad differentiates */
    RDF_OP_REM,          /* a, b -> remainder of the truncating division a / b (sign of a); 0 when b == 0 */
    /* Recursion driven by vector values (Section 6.2, last paragraph: a structure generated top-down by the model).
     * A program that uses one of the three operators below is executed with token scheduling and vector operators
     * interleaved wave by wave, because its Switches read states: fp32, RDF_TAGS_FRAME, rdf_eval only, H <= 256.
     * In such programs a formal parameter may be vector-valued (a call passes the state on by reference). */
    RDF_OP_CHILD_L,      /* a = state -> tanh(W[:, 0:H] a + b): the state of a node's left child, from its own */
    RDF_OP_CHILD_R,      /* a = state -> tanh(W[:, H:2H] a + b): the right child                              */
    RDF_OP_GATE,         /* a = state -> integer 1 if W_s[0] . a + b_s[0] > 0 else 0 (fp32 arithmetic)        */
    RDF_OP__COUNT
} rdf_opcode;

typedef struct {
    int32_t op;          /* rdf_opcode */
    int32_t a, b, c;     /* operand expression indices within the same function, -1 if unused */
    int64_t imm;
} rdf_expr;

typedef enum { RDF_FN_FUNCTION = 0, RDF_FN_LOOP = 1 } rdf_function_kind;

typedef struct {
    const char*     name;        /* host, NUL-terminated, copied by rdf_graph_build */
    int32_t         n_params;    /* m formal parameters: 1 for `result`, 1..3 for the others; m > 1 needs
                                    RDF_TAGS_FRAME (UNSUPPORTED otherwise) */
    int32_t         n_exprs;
    const rdf_expr* exprs;       /* host, [n_exprs]; a DAG (no cycles) */
    int32_t         root;        /* index of the expression that is the function's output */
    /* A definition of kind RDF_FN_LOOP is a while-loop (Section 2.3, Figure 1) over m loop-carried variables, its
     * parameters: while `cond` holds, variable k takes the value of `next[k]`; when it fails the loop's value is `root`,
     * evaluated on the final values.  A CALL of it with the initial values stands for the loop at that place: in
     * the static graph one Enter / Merge / Switch / Next per variable and an Exit, tags <0:t> on entry and
     * <(n+1):t> per iteration; loops and calls share the tag stack (Section 5.1).  `cond` and `root` must not
     * contain calls; `next[k]` may (functions, recursive ones, other loops).  Integer values, RDF_TAGS_FRAME.
     * (RDF_FN_FUNCTION: cond and next are ignored.) */
    int32_t         kind;        /* rdf_function_kind */
    int32_t         cond;
    int32_t         next[3];
} rdf_function;

typedef enum { RDF_TAGS_PATH = 0, RDF_TAGS_FRAME = 1 } rdf_tag_mode;

typedef struct {
    int32_t             n_functions;
    const rdf_function* functions;   /* host, [n_functions] */
    int32_t             result;      /* index of the definition of `result` */
    /* Tag representation on the device.
     * RDF_TAGS_PATH : the label list itself, packed in 64 bits
     *                 [63:44] instance | [43:38] depth | [37:0] labels, `label_bits` each, innermost lowest.
     *                 Matching uses an open-addressing hash table keyed by the packed tag.
     * RDF_TAGS_FRAME: an interned frame id; a frame record holds the parent frame and the label
     *                 (the paper's own representation, Section 5.1).  Needed for deep recursion,
     *                 for vector-valued programs and for functions of several parameters. */
    int32_t             tag_mode;
} rdf_program;

typedef struct rdf_graph rdf_graph;      /* opaque, owned by the library */

/* Section 3 transformation + lowering for the device.  All inputs are host
 * memory and are not retained.  On success *out_graph must be released with
 * rdf_graph_free.  Errors: BAD_PROGRAM, BAD_ARG, UNSUPPORTED. */
int  rdf_graph_build(const rdf_program* prog, rdf_graph** out_graph);
void rdf_graph_free(rdf_graph* g);

/* The literal static graph after the transformation of Section 3, for
 * inspection: Call_i / Return_i nodes, entry Merge nodes, Switch/Merge of the
 * conditionals, control edges Call_i -> Return_i (and entry Merge -> constant,
 * Figure 3).  Arrays are host memory owned by the graph. */
typedef enum {
    RDF_NODE_IN = 0, RDF_NODE_OUT, RDF_NODE_CONST, RDF_NODE_OP, RDF_NODE_SWITCH,
    RDF_NODE_MERGE, RDF_NODE_ENTRY_MERGE, RDF_NODE_CALL, RDF_NODE_RETURN,
    RDF_NODE_ENTER, RDF_NODE_EXIT, RDF_NODE_NEXT      /* tagged iteration, Section 2.3 */
} rdf_node_kind;

typedef struct {
    int32_t kind;        /* rdf_node_kind */
    int32_t op;          /* rdf_opcode for RDF_NODE_OP, else -1 */
    int32_t label;       /* i of Call_i / Return_i (numbered per callee from 0), else -1 */
    int32_t func;        /* function the node belongs to (Call/Return: the caller) */
    int32_t param;       /* parameter index for IN / ENTRY_MERGE / CALL */
    int32_t n_in;        /* number of data inputs */
    int64_t value;       /* constant value */
} rdf_node;

typedef struct {
    int32_t src, src_port;   /* Switch: output 0 = true side, 1 = false side */
    int32_t dst, dst_port;   /* dst_port = -1 for a control edge */
    int32_t control;
} rdf_edge;

typedef struct {
    int32_t         n_nodes, n_edges;
    const rdf_node* nodes;
    const rdf_edge* edges;
    int32_t         n_labels;    /* call sites in the whole program (device label ids are global: 0..n_labels-1) */
    int32_t         label_bits;  /* bits per label in the packed path tag */
    int32_t         n_match;     /* operators with more than one tagged input (token-store users) */
    int32_t         n_code;      /* instructions in the lowered device program */
    /* host [n_labels], owned by the graph: for device label id g, the function it calls and the i of
     * its Call_i / Return_i in the per-callee numbering of Section 3 (a tag of the paper lists these i) */
    const int32_t*  label_callee;
    const int32_t*  label_local;
} rdf_graph_desc;

int rdf_graph_describe(const rdf_graph* g, rdf_graph_desc* out);

/* ------------------------------------------------------------------- batch */
typedef struct {
    int64_t        B;            /* independent instances; each starts with the empty tag */
    const int64_t* x;            /* device [B]: argument of `result` for integer programs, NULL for tree programs */
    const int32_t* tree_root;    /* device [B]: root node of each tree (tree programs; the argument of `result`) */
    int64_t        N;            /* tree nodes in the flat arrays below (0 for integer programs) */
    const int32_t* left;         /* device [N], -1 at a leaf */
    const int32_t* right;        /* device [N], -1 at a leaf */
    const int32_t* tok;          /* device [N], token id at leaves */
    const int32_t* label;        /* device [N], class of every node (rdf_grad / NODE_LOSS), may be NULL for rdf_eval */
    int64_t        max_invocations; /* capacity: upper bound on Call firings over the batch (tree programs: N) */
    int64_t        max_wave_tokens; /* capacity of one wave's token queue; 0 = max_invocations + B */
} rdf_batch;

/* Parameters of the tree networks: fp32, row-major, device.  `compute` picks
 * the arithmetic of the cell contraction: RDF_F32 = fp32 FMA; RDF_BF16 = bf16
 * operands (states and weights rounded to bf16) with fp32 accumulation. */
typedef enum { RDF_F32 = 0, RDF_BF16 = 1 } rdf_compute;

typedef struct {
    int32_t      compute;        /* rdf_compute */
    int32_t      H, D, V, n_classes;
    int32_t      reproducible;   /* rdf_grad with RDF_BF16 on the tensor-core path: 1 = the parameter gradients and the loss
                                    come out bit for bit the same on every call with the same inputs (the cells are put in
                                    an order that depends on the input alone -- by call depth, then by the argument of the
                                    invocation -- every floating-point sum has a fixed order, and the sums that many thread
                                    blocks contribute to are exact integer sums in fixed point).  Slower; 0 = sums by
                                    atomics in arrival order (equal up to rounding).  Invocations of one depth that share
                                    an argument (a node reached twice) keep their arrival order.  UNSUPPORTED elsewhere. */
    const float* E;              /* [V, D]                                          */
    const float* W;              /* TreeRNN [H, 2H]; TreeLSTM [5H, 2H] (i, f_l, f_r, o, u) */
    const float* b;              /* [H] or [5H]                                     */
    const float* W_x;            /* TreeLSTM leaf projection [3H, D] (i, o, u) or NULL */
    const float* b_x;            /* [3H] or NULL                                    */
    const float* W_s;            /* loss head [n_classes, H] or NULL                */
    const float* b_s;            /* [n_classes] or NULL                             */
} rdf_params;

/* One record per Call firing and one per Return firing, in no particular
 * order (optional; for parity checks of tags). */
typedef struct {
    uint64_t tag;        /* PATH: packed tag of the invocation; FRAME: its frame id in the low half; inside a loop the
                            high half holds the iteration counter of the loop frame (the tag <n:t> of Section 2.3) */
    int64_t  value;      /* kind 0: the argument; kind 1: the returned integer (vector programs: frame id of the state);
                            kinds 2-4: the first loop variable */
    uint32_t kind;       /* 0 = Call fired (tag after the push), 1 = Return fired (tag before the pop),
                            2 = Enter fired (tag after), 3 = Next fired (tag after), 4 = Exit fired (tag before) */
    uint32_t label;      /* i of Call_i / Return_i (global label id); loops: 255 */
    uint32_t parent;     /* FRAME: frame id of the enclosing context (the tag below this one); PATH: 0 */
    uint32_t instance;   /* FRAME: iteration counter of the enclosing context when that is a loop frame, else 0;
                            PATH: bits [63:44] of the tag */
} rdf_trace_rec;

typedef struct {
    int64_t*       y;            /* device [B]: integer results, or NULL */
    float*         h_root;       /* device [B, H]: root states, or NULL */
    float*         loss;         /* device [1]: summed loss (rdf_grad), or NULL */
    rdf_trace_rec* trace;        /* device [trace_capacity] or NULL */
    int64_t        trace_capacity;
    uint64_t*      trace_count;  /* device [1]: records written (may exceed capacity: the excess was dropped) */
} rdf_outputs;

typedef struct {                 /* all device, fp32, shapes of the parameters; overwritten, not accumulated */
    float *dE, *dW, *db, *dW_x, *db_x, *dW_s, *db_s;
} rdf_param_grads;

typedef struct {
    int32_t  status;             /* RDF_OK or the first RDF_ERR_* the device recorded */
    uint32_t waves;              /* scheduler waves run (forward) */
    uint32_t waves_backward;
    uint32_t max_wave_tokens;    /* widest wave */
    uint64_t invocations;        /* Call firings */
    uint64_t tokens;             /* tokens taken from the wave queues */
    uint64_t store_inserts;      /* operands parked in the token store */
    uint64_t store_matches;      /* firings completed by a match */
    uint64_t store_probes;       /* hash slots inspected (PATH mode) */
    uint32_t max_probe;          /* longest probe sequence */
    uint32_t max_depth;          /* deepest tag (PATH mode) */
    uint64_t cells;              /* batched cell firings */
    uint64_t leaves;             /* batched leaf firings */
    /* SM clock cycles spent by thread block 0.  Forward: token scheduling (scheduler kernel), batched
       operators (operator kernel), waiting at grid barriers (both).  Gradient kernel: per-invocation
       work, batched operand gradients, waiting at grid barriers. */
    uint64_t cycles_schedule, cycles_batch, cycles_barrier;
    uint64_t cycles_bwd_frames, cycles_bwd_batch, cycles_bwd_barrier;
    uint32_t kernel_launches;    /* kernels of the library that the last call launched (host count; memsets and copies excluded) */
    uint32_t clusters;           /* thread-block clusters that fired the cells of the last call (fp32 TreeRNN without a grid
                                    barrier); 0 = the grid-wide operator kernel did */
} rdf_stats;

/* Bytes of device scratch rdf_eval (want_grad = 0) or rdf_grad (1) needs for
 * this graph and batch shape (only the sizes in `in` and `params` are read). */
int rdf_workspace_bytes(const rdf_graph* g, const rdf_batch* in, const rdf_params* params,
                        int want_grad, size_t* bytes);

/* Forward evaluation of `result` on every instance of the batch (Section 5.1:
 * run the static graph until no token is left).  Outputs: y or h_root. */
int rdf_eval(rdf_graph* g, const rdf_batch* in, const rdf_params* params, rdf_outputs* out,
             void* workspace, size_t workspace_bytes, void* stream);

/* rdf_eval for callers that can neither pass a workspace nor allocate one.
 * (The paper has no counterpart: this is a packaging variant of rdf_eval.)
 *
 * Who needs it: code that runs where device allocation is off limits -- inside
 * a memory pool that has already handed out everything, in a plug-in whose host
 * forbids cudaMalloc after start-up, or on a latency path where an allocation
 * (which may synchronise the device) is not acceptable.  Such a caller still
 * owns and passes the inputs and outputs; only the scratch is taken care of.
 *
 * The scratch is a fixed array of RDF_NOALLOC_SCRATCH_BYTES (16 MiB) that is part
 * of the library image: every GPU that loads the library holds it until the
 * process ends.  A batch whose rdf_workspace_bytes(.., want_grad = 0, ..) exceeds
 * that size is refused with RDF_ERR_WORKSPACE_TOO_SMALL and nothing is launched;
 * use rdf_eval with a workspace of your own for such batches.
 *
 * The call performs no cudaMalloc / cudaFree and calls no allocating library
 * routine.  The first call on each device looks up the array's device address
 * (a runtime query, done once per device with that device current); make that
 * first call outside any stream capture.  All calls on a device share the one
 * array, which still holds the previous call's data: the call clears what must
 * start from zero on `stream` before its kernels run, but two calls that overlap
 * on the GPU (different streams, or different graphs used concurrently) race on
 * it -- keep calls to this entry point ordered on one stream per device.
 * The status word and the counters that rdf_last_status reports live in the same
 * array: read them before the next call to this entry point on that device (with
 * any graph), or they describe that later call.
 * Everything else (arguments, outputs) is as for rdf_eval. */
#define RDF_NOALLOC_SCRATCH_BYTES (16u << 20)
int rdf_eval_noalloc(rdf_graph* g, const rdf_batch* in, const rdf_params* params, rdf_outputs* out,
                     void* stream);

/* Forward + reverse mode (Section 4): forward values are retained per
 * invocation; the gradient pass re-enters every invocation under the tag its
 * forward Call_i created and accumulates parameter gradients over all
 * invocations.  Loss = sum over all invocations marked by NODE_LOSS of the
 * softmax cross-entropy of W_s h + b_s against label[node].
 * Limits: H <= 1024 and n_classes <= 8 (UNSUPPORTED / BAD_ARG otherwise). */
int rdf_grad(rdf_graph* g, const rdf_batch* in, const rdf_params* params, rdf_outputs* out,
             rdf_param_grads* grads, void* workspace, size_t workspace_bytes, void* stream);

/* Synchronises the stream of the last rdf_eval/rdf_grad on this graph and
 * copies the device status word and counters out (host struct). */
int rdf_last_status(rdf_graph* g, rdf_stats* s);

const char* rdf_strerror(int status);

/* The hash form of the token store (RDF_TAGS_PATH; Section 2.2: an operator fires when its inputs hold tokens with
 * the same tag -- the store is where the first operand waits for the second), for the following calls on this graph.
 *   probe_mode : RDF_PROBE_THREAD -- every thread probes linearly for its own key (default);
 *                RDF_PROBE_WARP   -- the threads of a warp that reach the store together probe for one key at a time,
 *                                    each looking at one of 32 consecutive slots (a coalesced 512-byte load and a ballot).
 *   hash_slots : slots per matching operator (rounded up to a power of two, at least 1024); 0 = the default,
 *                the power of two at or above rdf_batch.max_invocations.  Entries are never removed, so a run
 *                needs one slot per parked operand; a table that is too small reports RDF_ERR_STORE_FULL.
 * Results do not depend on either setting.  rdf_workspace_bytes reflects hash_slots. */
enum { RDF_PROBE_THREAD = 0, RDF_PROBE_WARP = 1 };
int rdf_set_store(rdf_graph* g, int probe_mode, long long hash_slots);

/* Limits of the device executor for the following calls on this graph (the paper's
 * executor simply runs until both queues are empty, Section 5.1; these guards have
 * no counterpart there).
 *   wait_cycles : SM clock cycles a device-side wait (grid barrier, mbarrier) may last before the
 *                 kernel gives up with RDF_ERR_TIMEOUT; 0 restores the default (about two seconds).
 *   wave_limit  : scheduler waves a call may run before it stops with RDF_ERR_WAVE_LIMIT (the
 *                 guard against recursion that never reaches a base case); 0 restores the
 *                 default (2^24 for integer programs, twice the frame capacity for tree programs).
 * A call that ends with either status leaves the graph usable: the next call starts clean. */
int rdf_set_limits(rdf_graph* g, long long wait_cycles, long long wave_limit);

/* Measurement aid (the paper reports only wall-clock times, Section 6; there is
 * no counterpart to cite): when enabled, rdf_eval / rdf_grad record CUDA events
 * on their stream between the phases of a call.  rdf_last_phase_ms synchronises
 * those events and writes up to `capacity` durations in milliseconds to the
 * host array `ms`, in this order:
 *   0 set-up (clears, program upload, seed tokens, weight packing)
 *   1 scheduler waves (tokens: tag push / pop, matching, lists of ready operators)
 *   2 grouping of the ready cells by height     3 operator waves (batched leaves and cells)
 *   4 root states to the caller's buffer        5 loss head with dW_s, db_s
 *   6 lists of the gradient pass                7 gradient waves
 *   8 dW (and dW_x)   9 db   10 dE (TreeLSTM; the TreeRNN's dE is formed during the waves)
 * (rdf_eval fills 0..4).  *n receives the number written. */
enum { RDF_PHASE_SETUP = 0, RDF_PHASE_SCHEDULE, RDF_PHASE_GROUP, RDF_PHASE_OPERATORS, RDF_PHASE_ROOTS, RDF_PHASE_LOSS,
       RDF_PHASE_LISTS, RDF_PHASE_BACKWARD, RDF_PHASE_DW, RDF_PHASE_DB, RDF_PHASE_DE, RDF_PHASE__COUNT };
int rdf_set_profiling(rdf_graph* g, int enable);
int rdf_last_phase_ms(rdf_graph* g, float* ms, int capacity, int* n);

/* Measurement aid (no counterpart in the paper): the fp32 fused-multiply-add rate the current device reaches
 * on a register-resident loop, in TFLOP/s (host double) -- the peak the fp32 cell kernels are put against.
 * Runs a few short kernels on `stream` and synchronises them. */
int rdf_probe_fp32_fma(double* tflops, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* RDF_H */
