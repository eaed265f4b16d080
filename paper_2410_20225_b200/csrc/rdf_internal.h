// Internal structures shared by the host-side graph builder and the device
// executor.  Not part of the public boundary (see include/rdf.h).
#pragma once
#include <stdint.h>

#include <string>
#include <vector>

#include "rdf.h"

// ---------------------------------------------------------------------------
// Lowered device program.
//
// The static graph is cut into *segments*: maximal pieces that one arriving
// token (or one completed match) can run through without waiting for another
// token.  A segment is straight-line/branching code for a small register
// machine; the tag operations and the token-store accesses are instructions.
// ---------------------------------------------------------------------------
enum VmOp : uint8_t {
    VM_MOVI = 0,   // r[dst] = imm
    VM_MOVC,       // r[dst] = const_pool[imm]
    VM_MOV,        // r[dst] = r[a]
    VM_ADD, VM_SUB, VM_MUL, VM_MAX, VM_LT, VM_EQ, VM_REM,   // r[dst] = r[a] op r[b]
    VM_ISLEAF, VM_LEFT, VM_RIGHT, VM_TOK,           // r[dst] = tree accessor(r[a])
    VM_BRZ,        // Switch: if r[a] == 0 jump to imm (segment-relative before layout, absolute after)
    VM_JMP,        // jump to imm
    VM_CALL,       // Call_i: push label imm on the tag, send <i:t, r[a]> (further parameters r[b], r[dst]) to the callee
    VM_CALL_A,     // a Call_i that is followed in straight-line code by another one (VM_CALL_B): reserves frames and queue
    VM_CALL_B,     //   slots for both at once (one round of atomics on the token's critical path instead of two)
    VM_LDARG,      // r[dst] = parameter imm (> 0) of this invocation, kept in its frame
    VM_PORT,       // deliver r[a] to input port b of match node imm under the current tag
    VM_RET,        // the function's output r[a]: Return_i pops the tag and continues in the caller
    VM_OUT,        // r[a] is the program's output for this instance
    VM_EMBED,      // leaf state: queue E[r[a]] -> state of this frame; continue at segment imm next wave
    VM_LEAF_LSTM,  // same for the TreeLSTM leaf
    VM_ENTER,      // Enter: new loop frame under the current tag, counter 0; variables r[a], r[b], r[dst]; loop head at imm
    VM_NEXT,       // Next: counter + 1, variables r[a], r[b], r[dst], back to the loop head at imm (next wave)
    VM_EXIT,       // Exit: the tag below the loop frame again; carries on in the same segment
    VM_VCHILD,     // unary vector operator dst (0 left, 1 right half of W) on the state r[a] -> state of this frame; continue at imm next wave
    VM_VGATE,      // r[dst] = W_s[0] . state(r[a]) + b_s[0] > 0: an integer read off a vector value
    VM_HALT
};

struct VmInstr {
    uint8_t op, dst, a, b;
    int32_t imm;
};

enum MatchKind : int32_t { MATCH_INT = 0, MATCH_CELL_RNN = 1, MATCH_CELL_LSTM = 2 };

struct MatchNode {
    int32_t n_ports;     // tagged inputs that must meet
    int32_t kind;        // MatchKind
    int32_t cont_pc;     // INT: code run with r0..r(n-1) = port values; CELL_*: code run next wave with r0 = state slot
    int32_t port_base;   // first port in the dense (frame-mode) port array
};

enum ContKind : int32_t { K_PORT = 0, K_SEG = 1, K_RET = 2 };

struct LabelInfo {
    int32_t entry_pc;    // entry segment of the callee
    int32_t k_kind;      // what Return_i feeds: ContKind
    int32_t k_node;      // K_PORT: match node
    int32_t k_port;      // K_PORT: its port
    int32_t k_pc;        // K_SEG: code run with r0 = returned value
    int32_t child_index; // position of this call site among the call sites of its caller's body
    int32_t callee;      // function index
    int32_t local_label; // i of Call_i in the per-callee numbering of Section 3
    int32_t n_args;      // formal parameters of the callee (one Call_i node per parameter)
};

static const int RDF_MAX_REGS = 16;
static const int RDF_MAX_LABELS = 64;
static const int RDF_MAX_MATCH = 16;
static const int RDF_MAX_CODE = 1024;
static const int RDF_MAX_CONSTS = 64;
static const int RDF_PATH_BITS = 38;       // packed path field
static const int RDF_DEPTH_SHIFT = 38;     // 6-bit depth field above it
static const int RDF_INST_SHIFT = 44;      // 20-bit instance field

struct rdf_graph {
    // literal graph (Section 3 transformation), for inspection
    std::vector<rdf_node> nodes;
    std::vector<rdf_edge> edges;
    // lowered program
    std::vector<VmInstr> code;
    std::vector<MatchNode> match;
    std::vector<LabelInfo> labels;
    std::vector<int64_t> consts;
    std::vector<int32_t> label_callee, label_local;   // the same two fields of `labels`, as plain arrays for rdf_graph_describe
    int32_t result_entry_pc = 0;
    int32_t n_ports_total = 0;
    int32_t max_calls_per_body = 1;
    int32_t max_params = 1;
    int32_t label_bits = 1;
    int32_t tag_mode = RDF_TAGS_PATH;
    bool has_vector_ops = false;
    bool has_rnn = false, has_lstm = false, has_loss = false;
    bool uses_tree = false;
    bool has_loops = false;
    bool interleaved = false;     // some Switch reads a vector value: operators run between the token waves
    std::vector<std::string> func_names;
    // per-run state owned by the executor (rdf_exec.cu)
    void* dev = nullptr;
};

// implemented in rdf_exec.cu
void rdf_exec_release(rdf_graph* g);
