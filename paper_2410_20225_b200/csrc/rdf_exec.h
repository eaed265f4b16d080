// Shared between the forward executor (rdf_exec.cu) and the gradient pass
// (rdf_grad.cu): workspace layout, per-graph host state, the fp32 tile step.
#pragma once
#include <vector>
#include "rdf_device.cuh"

// ---- fp32 tiled contraction: 64 x 64 output tile, 16-deep steps, 256 threads, 4 x 4 per thread
static const int TM = 64, TN = 64, TK = 16;

// read and written with 128-bit accesses: rows are 272 bytes, the struct must sit on a 16-byte boundary
struct __align__(16) GemmSmem {
    float As[TK][TM + 4];     // [k][row of the tile]
    float Bs[TK][TN + 4];     // [k][column of the tile]
};

// TreeLSTM tiles: the same 64 x 64 tile for up to five gate blocks at once, so that all gates of a
// hidden unit end up in one thread and the gate arithmetic fuses into the epilogue
struct __align__(16) LstmSmem {
    float As[TK][TM + 4];
    float Bs[5][TK][TN + 4];
};

__device__ __forceinline__ float4 ldcg4(const float* p) { return __ldcg(reinterpret_cast<const float4*>(p)); }

__device__ __forceinline__ void gemm_tile_step(const GemmSmem& sm, int tx, int ty, float (&acc)[4][4]) {
#pragma unroll
    for (int kk = 0; kk < TK; ++kk) {
        const float4 av = *reinterpret_cast<const float4*>(&sm.As[kk][ty * 4]);
        const float4 bv = *reinterpret_cast<const float4*>(&sm.Bs[kk][tx * 4]);
        const float aa[4] = {av.x, av.y, av.z, av.w}, bb[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(aa[i], bb[j], acc[i][j]);
    }
}

// fp32 TreeRNN, narrow waves: a block keeps its 16 (forward) / 32 (gradient) columns of W in shared memory,
// 128 * H bytes, while that fits beside the tiles
static const int THIN_RESIDENT_MAX_H = 384;
inline size_t thin_resident_bytes(int lstm, int H) { return !lstm && H <= THIN_RESIDENT_MAX_H ? (size_t)128 * H : 0; }

static const int DW_BLOCKS_MAX = 256;        // blocks of the tensor-core weight-gradient pass (reproducible mode: one partial tile each)
static const int LIST_SEG = 2048;            // frames per segment of the list kernels (256 threads x 8)

// ---- host state
struct ExecState {
    int device = -1;
    int grid = 0;
    int last_clusters = 0;       // clusters the last call used
    int rnn32_per_sm = 1;        // blocks per SM of the fp32 TreeRNN operator / gradient kernels
    int n_clusters = 0;          // clusters of the clustered fp32 operator kernel that fit the device at once (0: none)
    int clock_khz = 0;
    void* last_ctl = nullptr;
    cudaStream_t last_stream = nullptr;
    bool ran = false;
    unsigned launches = 0;       // kernels launched by the last call
    int probe_mode = 0;          // rdf_set_store
    long long hash_slots = 0;
    long long wait_cycles = 0;   // rdf_set_limits: 0 = default
    long long wave_limit = 0;
    // optional phase timing
    bool profiling = false;
    cudaEvent_t ev[RDF_PHASE__COUNT + 1] = {};
    bool have_events = false;
    int n_phases = 0;
    // the lowered program (code, match nodes, labels, constants) as one block with the workspace's own spacing, so that
    // every call copies it to the device in one piece
    char*  tables = nullptr;     // the program tables as they lie in the workspace, in page-locked host memory (one async copy per call)
    size_t tables_bytes = 0;
    bool   tables_pinned = false;
    bool   may_allocate = true;  // false while rdf_eval_noalloc runs: the tables then stay in ordinary host memory
};

// records the boundary after phase `k - 1` (k = 0: start of the call)
inline void rdf_mark(ExecState* S, int k, cudaStream_t stream) {
    if (S->profiling && S->have_events) {
        cudaEventRecord(S->ev[k], stream);
        S->n_phases = k;
    }
}

struct Layout {
    size_t ctl, code, match, labels, consts, q0, q1, frames, frame_args, frame_ptag, finst, pair_slots, port_val, arrived, table, cell_items,
        leaf_items, cell_sorted, height_ends, op_l, op_r, arena, gates, arena_bf, wp, wtp, dz_bf, z_bf, zdst, cell_pos, wxp, wxtp, e_bf, dg_bf, ybuf, dhp, dlog, wave_marks, list_seg, all_cells, cell_ops, leaf_ops, all_leaves, loss_partial, dw_partial, de_fix, head_fix, rank_tmp, node_info, canon_hist, total;
    uint32_t qcap, frame_cap, work_cap, wave_cap, cells_cap, canon_cap;
    int use_tc, Hp, tc_smem_fwd, tc_smem_bwd, want_grad, repro, clustered;
    uint64_t table_cap;
    size_t arrived_bytes, table_bytes, pair_bytes;
};

// a kernel launch of the library, counted per call (rdf_stats.kernel_launches)
#define RDF_KERNEL(S, ...)  \
    do {                    \
        __VA_ARGS__;        \
        ++(S)->launches;    \
    } while (0)

#define CUDA_OK(expr)                                  \
    do {                                               \
        cudaError_t e_ = (expr);                       \
        if (e_ != cudaSuccess) return RDF_ERR_CUDA;    \
    } while (0)

int rdf_make_layout(const rdf_graph* g, const rdf_batch* in, const rdf_params* params, int want_grad, Layout& L);
ExecState* rdf_state_of(rdf_graph* g);
int rdf_prepare_device(rdf_graph* g, ExecState* S);
void rdf_fill_ctx(rdf_graph* g, const rdf_batch* in, const rdf_params* params, rdf_outputs* out, char* ws,
                  const Layout& L, ExecState* S, DevCtx& c);
int rdf_check_common(rdf_graph* g, const rdf_batch* in, const rdf_params* params, rdf_outputs* out, void* ws);
// a row-major bf16 matrix [rows, cols] as a 2D tensor map for tile copies: boxes of box_rows x 64 columns, 128-byte swizzle
int encode_row_tiles(TensorMap* out, void* base, uint64_t rows, uint64_t cols, uint32_t box_rows);
// the lists over the frames (cells in depth order, waves, operand-row destinations); TC path: part of the forward pass
int rdf_launch_depth_groups(char* ws, const Layout& L, ExecState* S, DevCtx& c, cudaStream_t stream);
int rdf_launch_lists(const rdf_batch* in, char* ws, const Layout& L, ExecState* S, DevCtx& c, cudaStream_t stream);
int rdf_launch_forward(rdf_graph* g, const rdf_batch* in, rdf_outputs* out, char* ws, const Layout& L, ExecState* S,
                       DevCtx& c, cudaStream_t stream);
