// Tensor-core path (sm_100a: tcgen05 + tensor memory) for the dense
// contractions of the bf16 workloads, forward and operand-gradient:
//
//   forward :  D[128 cells x NS] = A[128 x 2Hp] * Wp [NS x 2Hp]^T     A row = [h_l ; h_r] (bf16 states, gathered)
//   backward:  D[128 cells x NS] = A[128 x  Hp] * WTp[NS x  Hp]^T     A row = dz (bf16),  D = slice of [dh_l ; dh_r]
//
// Weight-stationary: the packed weight matrix is split along N into slices; a
// thread block owns one slice for the whole kernel and keeps it in shared
// memory (loaded once, <= 130 KB), so per tile only the gathered operand rows
// move.  The tile loop is a pipeline of three roles inside the 416-thread block:
//   producers (4 warps): gather the operand rows with cp.async into a ring of 128-byte-swizzled
//       [128 x 64] bf16 stages (8-row groups of 1024 bytes, 16-byte chunks XOR-ed with the row index:
//       the K-major layout the MMA reads), several stages ahead and across tile boundaries;
//   MMA issuer (1 thread): tcgen05.mma per stage into one of two accumulator buffers in tensor
//       memory; tcgen05.commit frees the stage and, after a tile's last stage, publishes the buffer;
//   epilogue (8 warps): tcgen05.ld of a finished buffer, bias / activations, stores -- while the
//       MMAs of the next tile fill the other buffer.
// The roles meet only through mbarriers, and every wait is bounded.
#pragma once
#include <cuda_bf16.h>

#include "rdf_exec.h"

static const int TC_M = 128;                 // cells per tile (TMEM lanes)
static const int TC_KC = 64;                 // bf16 elements per staged K chunk = one 128-byte swizzled row
static const int TC_MAX_STAGES = 8;
static const int TC_A_STAGE = TC_M * 128;    // 16 KB
static const int TC_HP_MAX = 320;            // widest padded hidden size the resident slices are sized for
static const int TC_ACC_COLS = 128;          // TMEM columns per accumulator buffer
static const int TC_TMEM_COLS = 2 * TC_ACC_COLS;
static const int TC_THREADS = 416;           // warps 0-7 epilogue, warp 8 MMA issuer, warps 9-12 producers
static const int TC_EPI_THREADS = 256, TC_MMA_WARP = 8, TC_PROD_WARP0 = 9, TC_PRODUCERS = 128;
// ring depth per kernel: what is left of the shared memory beside the resident weight slices
static const int TC_STAGES_RNN_FWD = 7, TC_STAGES_LSTM_FWD = 5, TC_STAGES_RNN_BWD = 8, TC_STAGES_LSTM_BWD = 4;
// TreeLSTM operand gradient: columns of WT5p per block.  Every block of a row group gathers the same operand rows, so
// the wider the slice the fewer copies of them cross L2; 48 columns x 5 Hp is what fits beside a ring of 4 stages.
static const int TC_LSTM_BWD_NS = 48;

// tile loops (template parameter of tc_pipe)
enum TcMode {
    TC_RNN_FWD = 0,     // A = [h_l ; h_r] (operand rows), B = Wp slice;           epilogue: tanh, bf16 state
    TC_RNN_BWD = 1,     // A = dz,                         B = WTp slice;          epilogue: dz of the callee cells, dE of the callee leaves
    TC_LSTM_CELL = 2,   // A = [h_l ; h_r],                B = W5p slice (5 gates x 16 units); epilogue: gates, c, h
    TC_LSTM_LEAF = 3,   // A = E_bf[tok],                  B = Wxp slice (3 gates x 16 units); epilogue: gates, c, h
    TC_LSTM_BWD = 4,    // A = gate gradients (5 Hp),      B = WT5p slice;         epilogue: operand gradients (dh)
    TC_LSTM_DE = 5      // A = leaf gate gradients (3 Hp), B = WxTp slice;         epilogue: dE[tok] += W_x^T dg
};

// mbarriers and tile records of the pipeline (static shared memory of the kernel)
struct __align__(16) TcShared {
    uint4    items[2][TC_M];                 // per accumulator buffer: {frame, left, right / token, valid} of the tile's rows
    uint64_t full[TC_MAX_STAGES];            // stage filled (all producer threads arrived)
    uint64_t empty[TC_MAX_STAGES];           // stage consumed (tcgen05.commit)
    uint64_t acc_full[2], acc_empty[2];      // accumulator buffer complete / read out by the epilogue
    uint64_t items_full[2];                  // tile records written
    uint32_t tmem_slot;
    // what the epilogue adds to this block's slice of columns, copied once per kernel (the 30 KB of L1 left
    // beside the operand stages do not keep it): TreeRNN forward: bias[col]; TreeLSTM: cell bias [gate][unit]
    // at 0, leaf bias at TC_EP_LEAF; TreeRNN gradient: W_s[class][col of the callee] (zero beyond H and C)
    __align__(16) float ep[8 * (TC_HP_MAX / 4)];       // read with 128-bit loads
};
struct TcState {
    uint32_t tmem_base;      // TMEM address returned by tcgen05.alloc
    uint32_t a_addr;         // shared-space address of A stage 0
    uint32_t g;              // K chunks that went through the ring so far (stage = g % stages)
    uint32_t T;              // tiles this block has run so far (accumulator buffer = T % 2)
    int      n_split;        // N slices = blocks per row group
    // up to two resident weight slices (the TreeLSTM forward keeps the cell and the leaf weights)
    uint32_t b_addr[2];
    int      ns[2], n_chunks[2];
};

static const int TC_EP_LD = TC_HP_MAX / 4, TC_EP_LEAF = 5 * 16;

// Fills TcShared::ep for the kernel's mode (all threads call it, after tc_setup).
__device__ __forceinline__ void tc_setup_epilogue(const DevCtx& c, const TcState& tc, TcShared& sh, bool gradient) {
    const int H = c.H, Hp = c.Hp, slice = blockIdx.x % tc.n_split;
    for (int q = threadIdx.x; q < 8 * TC_EP_LD; q += blockDim.x) {
        float v = 0.f;
        const int k = q / TC_EP_LD, j = q % TC_EP_LD;
        if (gradient) {                                   // W_s[k][column of the callee]
            const int col = slice * tc.ns[0] + j, cc = col < Hp ? col : col - Hp;
            if (!c.lstm && j < tc.ns[0] && k < c.n_classes && cc < H) v = c.W_s[k * H + cc];
        } else if (c.lstm) {                              // [gate][unit] of the slice's 16 units
            const int g = q / 16, u = slice * 16 + q % 16;
            if (q < TC_EP_LEAF) { if (u < H) v = c.b[g * H + u]; }
            else if (q < TC_EP_LEAF + 48) { if (u < H) v = c.b_x[(g - 5) * H + u]; }
        } else if (k == 0) {
            const int col = slice * tc.ns[0] + j;
            if (j < tc.ns[0] && col < H) v = c.b[col];
        }
        sh.ep[q] = v;
    }
    __syncthreads();
}

// dynamic shared memory a kernel needs for the given resident slices and ring depth
inline int tc_smem_bytes(int ns0, int k0, int ns1, int k1, int stages) {
    return 1024 + (k0 / TC_KC) * ns0 * 128 + (ns1 ? (k1 / TC_KC) * ns1 * 128 : 0) + stages * TC_A_STAGE;
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t addr, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(addr), "r"(count) : "memory");
}

// Bounded wait for the phase with the given parity.  Returns false on expiry.
__device__ __forceinline__ bool mbar_wait(const DevCtx& c, uint32_t addr, uint32_t parity) {
    const long long t0 = clock64();
    for (uint32_t polls = 0;; ++polls) {
        uint32_t done;
        asm volatile(
            "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
            : "=r"(done) : "r"(addr), "r"(parity) : "memory");
        if (done) return true;
        if (clock64() - t0 > c.spin_limit) {
            set_status(c, RDF_ERR_TIMEOUT);
            return false;
        }
        // a role that gave up elsewhere (any block) will not complete this phase: leave with it
        if ((polls & 255u) == 255u && ld_volatile_i32(&c.ctl->status) != 0) return false;
    }
}

// Shared-memory operand descriptor: K-major, 128-byte swizzle, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t tc_desc(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);       // start address, 16-byte units
    d |= (uint64_t)1 << 16;                              // leading byte offset (unused for this layout)
    d |= (uint64_t)(1024 >> 4) << 32;                    // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;                              // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                              // 128-byte swizzle
    return d;
}

// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N given.
__device__ __forceinline__ uint32_t tc_idesc(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(TC_M >> 4) << 24);
}

__device__ __forceinline__ void tc_mma(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
        " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}

__device__ __forceinline__ void tc_commit(uint32_t mbar_addr) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(mbar_addr) : "memory");
}

__device__ __forceinline__ void tc_ld16(uint32_t taddr, float (&v)[16]) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];\n"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// the same without the wait: several loads in flight, then one tc_wait_ld()
__device__ __forceinline__ void tc_ld16_issue(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];\n"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// 32 contiguous bytes in one store (a whole sector per lane: half the requests of two 16-byte stores);
// the address is 32-byte aligned
__device__ __forceinline__ void st_global_32(void* p, const uint4& a, const uint4& b) {
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(p), "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w),
                 "r"(b.x), "r"(b.y), "r"(b.z), "r"(b.w) : "memory");
}

// 16-byte asynchronous copy global -> shared through L2; `valid == false` writes zeros
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
    const int n = valid ? 16 : 0;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(n) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
// the same with a run-time count (the instruction takes an immediate)
__device__ __forceinline__ void cp_async_wait_upto(uint32_t n) {
    switch (n) {
        case 0: cp_async_wait<0>(); break;
        case 1: cp_async_wait<1>(); break;
        case 2: cp_async_wait<2>(); break;
        case 3: cp_async_wait<3>(); break;
        case 4: cp_async_wait<4>(); break;
        case 5: cp_async_wait<5>(); break;
        default: cp_async_wait<6>(); break;
    }
}

// byte offset of 16-byte chunk c16 of row r inside a swizzled [rows x 128 bytes] operand tile
__device__ __forceinline__ uint32_t swz(int r, int c16) {
    return (uint32_t)((r >> 3) * 1024 + (r & 7) * 128 + ((c16 ^ (r & 7)) << 4));
}

// The executing thread arrives on the mbarrier once all cp.async copies it has issued so far have landed
// (the barrier's count already includes this arrival).
__device__ __forceinline__ void cp_async_arrive(uint32_t mbar_addr) {
    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(mbar_addr) : "memory");
}

// One box of a 2D tensor map (tile mode) into shared memory; completion is counted in bytes on the mbarrier.
// x (innermost coordinate) times the element size must be a multiple of 16 bytes.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const TensorMap* map, int x, int y, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t addr, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(addr), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t addr, uint32_t bytes) {
    asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(addr), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t addr) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(addr) : "memory");
}

// One-time set-up per kernel (all threads call it): TMEM allocation by warp 0, mbarriers, and the
// block's resident slices of the packed weights: rows [slice * ns, +ns) of B[. x K], chunk by chunk.
__device__ __forceinline__ void tc_setup(TcState& tc, TcShared& sh, unsigned char* dyn_smem, int n_split,
                                         const __nv_bfloat16* B0, int K0, int ns0,
                                         const __nv_bfloat16* B1 = nullptr, int K1 = 0, int ns1 = 0, int rows0 = 1 << 30) {
    // (rows0: rows of B0 that exist; the last slice may reach beyond them and holds zeros there)
    const uint32_t raw = smem_u32(dyn_smem);
    const uint32_t aligned = (raw + 1023u) & ~1023u;
    unsigned char* base = dyn_smem + (aligned - raw);
    const int bytes0 = (K0 / TC_KC) * ns0 * 128, bytes1 = B1 ? (K1 / TC_KC) * ns1 * 128 : 0;
    tc.b_addr[0] = aligned;
    tc.b_addr[1] = aligned + bytes0;
    tc.a_addr = aligned + bytes0 + bytes1;
    tc.ns[0] = ns0; tc.ns[1] = ns1;
    tc.n_chunks[0] = K0 / TC_KC; tc.n_chunks[1] = B1 ? K1 / TC_KC : 0;
    tc.g = 0;
    tc.T = 0;
    tc.n_split = n_split;
    if (threadIdx.x == 0) {
        for (int s = 0; s < TC_MAX_STAGES; ++s) {
            mbar_init(smem_u32(&sh.full[s]), TC_PRODUCERS);
            mbar_init(smem_u32(&sh.empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&sh.acc_full[b]), 1);
            mbar_init(smem_u32(&sh.acc_empty[b]), TC_EPI_THREADS);
            mbar_init(smem_u32(&sh.items_full[b]), TC_PRODUCERS);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (threadIdx.x < 32) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh.tmem_slot)), "n"(TC_TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    const int slice = blockIdx.x % n_split;
    for (int which = 0; which < 2; ++which) {
        const __nv_bfloat16* Bp = which ? B1 : B0;
        if (!Bp) continue;
        const int ns = which ? ns1 : ns0, Kp = which ? K1 : K0;
        unsigned char* bp = base + (which ? bytes0 : 0);
        for (int p = threadIdx.x; p < (Kp / TC_KC) * ns * 8; p += blockDim.x) {
            const int kc = p / (ns * 8), q = p % (ns * 8), r = q >> 3, c16 = q & 7;
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            if (which || slice * ns + r < rows0) v = *reinterpret_cast<const uint4*>(Bp + (size_t)(slice * ns + r) * Kp + kc * TC_KC + c16 * 8);
            *reinterpret_cast<uint4*>(bp + kc * ns * 128 + swz(r, c16)) = v;
        }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    tc.tmem_base = *reinterpret_cast<volatile uint32_t*>(&sh.tmem_slot);
}

__device__ __forceinline__ void tc_teardown(const TcState& tc) {
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (threadIdx.x < 32)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tc.tmem_base), "n"(TC_TMEM_COLS) : "memory");
}

__device__ __forceinline__ void tc_ld8(uint32_t taddr, float (&v)[8]) {
    uint32_t r[8];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];\n"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
        : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(r[i]);
}

// Activations of the bf16 path: one MUFU instruction each (relative error about 2^-11, below the bf16
// rounding of the operands they feed).
__device__ __forceinline__ float tc_tanh(float x) {
    float y;
    asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float tc_sigmoid(float x) { return fmaf(0.5f, tc_tanh(0.5f * x), 0.5f); }

// The tile loop over n_items ready operators (see TcMode), 128 rows per tile.  Rows come from
// cell_items / leaf_items (forward modes) or from cell_ops / leaf_ops at [first ..] (gradient modes).
// Called by all TC_THREADS threads of the block; returns when every tile has been written out.
template <int MODE, int STAGES>
__device__ void tc_pipe(const DevCtx& c, TcState& tc, TcShared& sh, uint32_t first, uint32_t n_items) {
    static_assert(STAGES >= 3 && STAGES <= TC_MAX_STAGES, "ring depth");
    constexpr int RGN = MODE == TC_LSTM_LEAF ? 1 : 0;
    // The rows of the A operand are consecutive rows of a matrix (the operand rows z_bf of the listed cells, or their
    // dz rows): one 2D tile copy per stage instead of a gather.
    constexpr bool TMA_A = MODE == TC_RNN_FWD || MODE == TC_LSTM_CELL || MODE == TC_RNN_BWD;
    // These modes write rows that later tile copies read (states into operand rows, dz rows).
    constexpr bool WRITES_TILE_ROWS = MODE == TC_RNN_FWD || MODE == TC_LSTM_CELL || MODE == TC_LSTM_LEAF || MODE == TC_RNN_BWD;
    const int H = c.H, Hp = c.Hp, S = c.S, ns = tc.ns[RGN], n_chunks = tc.n_chunks[RGN];
    const int slice = blockIdx.x % tc.n_split, rg = blockIdx.x / tc.n_split, n_rg = gridDim.x / tc.n_split;
    const int tiles = (n_items + TC_M - 1) / TC_M;
    // blocks beyond the last full group of slices have no tiles
    const int my_tiles = rg < n_rg && tiles > rg ? (tiles - rg + n_rg - 1) / n_rg : 0;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t full0 = smem_u32(&sh.full[0]), empty0 = smem_u32(&sh.empty[0]);
    const uint32_t acc_full0 = smem_u32(&sh.acc_full[0]), acc_empty0 = smem_u32(&sh.acc_empty[0]);
    const uint32_t items_full0 = smem_u32(&sh.items_full[0]);
    bool ok = true;
    if (warp >= TC_PROD_WARP0) {
        // ------------------------------------------------------------ producers
        const int p = threadIdx.x - TC_PROD_WARP0 * 32, r8 = p >> 3, c16 = p & 7;
        const __nv_bfloat16* Arows = (MODE == TC_LSTM_BWD || MODE == TC_LSTM_DE) ? c.dg_bf
                                     : MODE == TC_LSTM_LEAF ? c.E_bf : c.arena_bf;
        auto load_item = [&](int tile) {                     // the record of row p of the tile
            uint4 it = make_uint4(0u, 0u, 0u, 0u);
            const uint32_t row = (uint32_t)tile * TC_M + p;
            if (row < n_items) {
                if (MODE == TC_LSTM_DE) it = __ldcg(&c.leaf_ops[first + row]);                   // {leaf frame, token id, -, 1}
                else if (MODE == TC_LSTM_LEAF) {
                    const uint2 lf = __ldcg(reinterpret_cast<const uint2*>(&c.leaf_items[first + row]));     // {slot, tok}
                    it.x = lf.x; it.y = lf.y;
                } else it = __ldcg(&c.cell_ops[first + row]);                                    // {cell, left, right, 1}
                it.w = 1u;
            }
            return it;
        };
        // the rows the tiles read were written with plain stores by other blocks before the last grid barrier: order
        // this call's tile copies (async proxy) after what that barrier acquired
        if (TMA_A) asm volatile("fence.proxy.async;" ::: "memory");
        uint4 it_next = my_tiles ? load_item(rg) : make_uint4(0u, 0u, 0u, 0u);
        for (int i = 0; i < my_tiles && ok; ++i) {
            const uint32_t T = tc.T + i, b = T & 1u;
            // the epilogue of the tile before last has finished with this record buffer
            if (T >= 2) ok = mbar_wait(c, acc_empty0 + 8 * b, ((T >> 1) - 1) & 1u);
            sh.items[b][p] = it_next;
            mbar_arrive(items_full0 + 8 * b);
            if (i + 1 < my_tiles) it_next = load_item(rg + (i + 1) * n_rg);      // in flight during this tile
            ok = mbar_wait(c, items_full0 + 8 * b, (T >> 1) & 1u) && ok;
            // the eight rows this thread copies: r8 + 16 q
            uint32_t src0[8], src1[8], valid = 0;
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                const uint4 it = sh.items[b][r8 + 16 * q];
                if (it.w) valid |= 1u << q;
                if (MODE == TC_RNN_FWD || MODE == TC_LSTM_CELL) { src0[q] = it.y; src1[q] = it.z; }
                else if (MODE == TC_LSTM_LEAF) { src0[q] = it.y; src1[q] = it.y; }
                else { src0[q] = it.x; src1[q] = it.x; }
            }
            const size_t lda = (MODE == TC_LSTM_BWD || MODE == TC_LSTM_DE) ? (size_t)5 * Hp : (size_t)Hp;
            for (int kc = 0; kc < n_chunks && ok; ++kc) {
                const uint32_t g = tc.g + (uint32_t)(i * n_chunks + kc), s = g % STAGES;
                // the MMAs that last read this stage must have completed
                if (g >= (uint32_t)STAGES) ok = mbar_wait(c, empty0 + 8 * s, ((g / STAGES) - 1) & 1u);
                if (TMA_A) {
                    // the rows of the wave's cells are consecutive: one 2D tile (128 rows x 64 columns, written in the
                    // 128-byte swizzle by the copy engine) per stage.  Rows after the wave's last cell hold other cells'
                    // rows or old data: their accumulator rows are never read.
                    if (!ok) break;
                    if (p == 0) {
                        mbar_arrive_expect_tx(full0 + 8 * s, TC_A_STAGE);
                        tma_load_2d(tc.a_addr + s * TC_A_STAGE, MODE == TC_RNN_BWD ? &c.tmap_dz128 : &c.tmap_z128, kc * TC_KC,
                                    (int)(first + (uint32_t)(rg + i * n_rg) * TC_M), full0 + 8 * s);
                    } else mbar_arrive(full0 + 8 * s);
                    continue;
                }
                const int koff = kc * TC_KC;
                const bool second = (MODE == TC_RNN_FWD || MODE == TC_LSTM_CELL) && koff >= Hp;
                const size_t col = (size_t)(second ? koff - Hp : koff) + c16 * 8;
#pragma unroll
                for (int q = 0; q < 8; ++q)
                    cp_async16(tc.a_addr + s * TC_A_STAGE + swz(r8 + 16 * q, c16),
                               Arows + (size_t)(second ? src1[q] : src0[q]) * lda + col, (valid >> q) & 1u);
                cp_async_arrive(full0 + 8 * s);                // this thread's share of the stage: arrives when its copies have landed
            }
        }
    } else if (warp == TC_MMA_WARP) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc = tc_idesc(ns);
            for (int i = 0; i < my_tiles && ok; ++i) {
                const uint32_t T = tc.T + i, b = T & 1u;
                // the epilogue has read the previous contents of this accumulator buffer
                if (T >= 2) ok = mbar_wait(c, acc_empty0 + 8 * b, ((T >> 1) - 1) & 1u);
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                for (int kc = 0; kc < n_chunks && ok; ++kc) {
                    const uint32_t g = tc.g + (uint32_t)(i * n_chunks + kc), s = g % STAGES;
                    ok = mbar_wait(c, full0 + 8 * s, (g / STAGES) & 1u);
                    if (!ok) break;
                    // a stage written by cp.async (generic proxy) is read by the MMA (async proxy); tile copies are async-proxy writes
                    if (!TMA_A) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t a = tc.a_addr + s * TC_A_STAGE, bw = tc.b_addr[RGN] + kc * ns * 128;
#pragma unroll
                    for (int ks = 0; ks < TC_KC / 16; ++ks)
                        tc_mma(tc.tmem_base + b * TC_ACC_COLS, tc_desc(a + ks * 32), tc_desc(bw + ks * 32), idesc,
                               (kc > 0 || ks > 0) ? 1u : 0u);
                    tc_commit(empty0 + 8 * s);                 // the stage is free when these MMAs have read it
                }
                if (ok) tc_commit(acc_full0 + 8 * b);          // the accumulators are complete when all MMAs so far are
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------ epilogue
        for (int i = 0; i < my_tiles && ok; ++i) {
            const uint32_t T = tc.T + i, b = T & 1u;
            ok = mbar_wait(c, items_full0 + 8 * b, (T >> 1) & 1u);
            if (!ok) break;
            const int row = (warp & 3) * 32 + lane;                       // warp w reads TMEM lanes 32 (w % 4) ..
            const uint32_t lane_base = tc.tmem_base + (uint32_t)(b * TC_ACC_COLS) + ((uint32_t)((warp & 3) * 32) << 16);
            const uint4 it = sh.items[b][row];
            const bool live = it.w != 0u;
            // TreeRNN gradient: what the epilogue needs about the callee frame is fetched while the MMAs run.
            // All columns of a slice belong to one callee: [0, Hp) to the left one, [Hp, 2Hp) to the right one.
            // Units of 8 columns, warps 0-3 take the first half of them and warps 4-7 the rest.
            constexpr int BWD_MAXU = (TC_HP_MAX / 4 / 8 + 1) / 2;
            const int e_units = ns / 8, e_lo = (e_units + 1) / 2;
            const int e_begin = warp < 4 ? 0 : e_lo, e_end = warp < 4 ? e_lo : e_units;
            const int e_col0 = slice * ns;
            const uint32_t child = e_col0 < Hp ? it.y : it.z;
            const int e_cc0 = e_col0 < Hp ? e_col0 : e_col0 - Hp;
            // forward modes: where this invocation's state goes besides its own row (the operand row of its caller)
            uint32_t zd = NO_ZDST;
            if ((MODE == TC_RNN_FWD || MODE == TC_LSTM_CELL || MODE == TC_LSTM_LEAF) && live) zd = __ldg(&c.zdst[it.x]);
            __nv_bfloat16* zrow = zd != NO_ZDST ? c.z_bf + (size_t)(zd >> 1) * 2 * Hp + (size_t)(zd & 1u) * Hp : nullptr;
            uint32_t child_l = LEAF_MARK, child_tok = 0, child_pos = 0;
            float4 cd0 = make_float4(0.f, 0.f, 0.f, 0.f), cd1 = cd0;
            uint4 chq[BWD_MAXU];
            if (MODE == TC_RNN_BWD && live) {
                child_l = c.op_l[child];
                child_tok = c.op_r[child];
                child_pos = c.cell_pos[child];                            // (a cell's dz row; meaningless for a leaf)
                cd0 = *reinterpret_cast<const float4*>(c.dlog + (size_t)child * 8);
                cd1 = *reinterpret_cast<const float4*>(c.dlog + (size_t)child * 8 + 4);
#pragma unroll
                for (int q = 0; q < BWD_MAXU; ++q)
                    if (e_begin + q < e_end)
                        chq[q] = *reinterpret_cast<const uint4*>(c.arena_bf + (size_t)child * Hp + e_cc0 + (e_begin + q) * 8);
            }
            ok = mbar_wait(c, acc_full0 + 8 * b, (T >> 1) & 1u);
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            if (MODE == TC_RNN_BWD) {
                // dh of the callee = its slice of W^T dz (the accumulators) + W_s^T dlog of the callee;
                // a cell callee gets dz = dh (1 - h^2) as its bf16 operand row for the next wave (and for dW),
                // a leaf callee adds dh to row tok of dE.  No gradient ever goes to memory in fp32.
                const float dl[8] = {cd0.x, cd0.y, cd0.z, cd0.w, cd1.x, cd1.y, cd1.z, cd1.w};
#pragma unroll
                for (int q = 0; q < BWD_MAXU; ++q) {
                    if (e_begin + q >= e_end) continue;                   // (uniform over the warp)
                    float v[8];
                    tc_ld8(lane_base + (uint32_t)((e_begin + q) * 8), v);
                    if (!live) continue;
                    const int cc = e_cc0 + (e_begin + q) * 8;
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        if (k >= c.n_classes) break;                      // (uniform)
                        const float* wk = &sh.ep[k * TC_EP_LD + (e_begin + q) * 8];
                        const float4 w0 = *reinterpret_cast<const float4*>(wk), w1 = *reinterpret_cast<const float4*>(wk + 4);
                        v[0] = fmaf(w0.x, dl[k], v[0]); v[1] = fmaf(w0.y, dl[k], v[1]);
                        v[2] = fmaf(w0.z, dl[k], v[2]); v[3] = fmaf(w0.w, dl[k], v[3]);
                        v[4] = fmaf(w1.x, dl[k], v[4]); v[5] = fmaf(w1.y, dl[k], v[5]);
                        v[6] = fmaf(w1.z, dl[k], v[6]); v[7] = fmaf(w1.w, dl[k], v[7]);
                    }
                    if (child_l == LEAF_MARK) {
                        if (c.dE_fix) {                               // reproducible mode: exact integer sums
                            long long* de = c.dE_fix + (size_t)child_tok * c.D + cc;
#pragma unroll
                            for (int i = 0; i < 8; ++i)
                                if (cc + i < H) fix_add(de + i, to_fix(v[i]));
                        } else {
                            float* de = c.dE + (size_t)child_tok * c.D + cc;
                            if (cc < H) atomicAdd(reinterpret_cast<float4*>(de), make_float4(v[0], v[1], v[2], v[3]));
                            if (cc + 4 < H) atomicAdd(reinterpret_cast<float4*>(de + 4), make_float4(v[4], v[5], v[6], v[7]));
                        }
                    } else {
                        __align__(16) __nv_bfloat162 pk[4];
                        const __nv_bfloat162* hb = reinterpret_cast<const __nv_bfloat162*>(&chq[q]);
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const float2 x = __bfloat1622float2(hb[i]);       // pad columns: v = 0, so dz = 0
                            pk[i] = __floats2bfloat162_rn(v[2 * i] * (1.f - x.x * x.x), v[2 * i + 1] * (1.f - x.y * x.y));
                        }
                        *reinterpret_cast<uint4*>(c.dz_bf + (size_t)child_pos * Hp + cc) = *reinterpret_cast<const uint4*>(pk);
                    }
                }
            } else if (MODE == TC_LSTM_CELL || MODE == TC_LSTM_LEAF) {
                // slice = 16 hidden units, columns gate * 16 + unit; warps 0-3 take units 0-7, warps 4-7 units 8-15
                constexpr int NG = MODE == TC_LSTM_CELL ? 5 : 3;
                const int wg = warp >> 2, u0 = slice * 16 + wg * 8;
                float v[NG][8];
#pragma unroll
                for (int g = 0; g < NG; ++g) tc_ld8(lane_base + (uint32_t)(g * 16 + wg * 8), v[g]);
                if (live) {
                    const float* bias = MODE == TC_LSTM_CELL ? sh.ep : sh.ep + TC_EP_LEAF;     // [gate][unit of the slice]
                    float cl[8], cr[8], hv[8], cv[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) cl[i] = cr[i] = 0.f;
                    if (MODE == TC_LSTM_CELL) {
#pragma unroll
                        for (int i = 0; i < 8; i += 4)
                            if (u0 + i < H) {
                                const float4 a = ldcg4(c.arena + (size_t)it.y * S + H + u0 + i);
                                const float4 b = ldcg4(c.arena + (size_t)it.z * S + H + u0 + i);
                                cl[i] = a.x; cl[i + 1] = a.y; cl[i + 2] = a.z; cl[i + 3] = a.w;
                                cr[i] = b.x; cr[i + 1] = b.y; cr[i + 2] = b.z; cr[i + 3] = b.w;
                            }
                    }
                    __align__(16) __nv_bfloat16 hb[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const int u = u0 + i;
                        float h = 0.f, cc = 0.f;
                        if (u < H) {
                            if (MODE == TC_LSTM_CELL) {
                                const float gi = tc_sigmoid(v[0][i] + bias[wg * 8 + i]);
                                const float fl = tc_sigmoid(v[1][i] + bias[16 + wg * 8 + i]);
                                const float fr = tc_sigmoid(v[2][i] + bias[32 + wg * 8 + i]);
                                const float go = tc_sigmoid(v[3 % NG][i] + bias[48 + wg * 8 + i]);
                                const float gu = tc_tanh(v[4 % NG][i] + bias[64 + wg * 8 + i]);
                                cc = gi * gu + fl * cl[i] + fr * cr[i];
                                h = go * tc_tanh(cc);
                                v[0][i] = gi; v[1][i] = fl; v[2][i] = fr; v[3 % NG][i] = go; v[4 % NG][i] = gu;
                            } else {
                                const float gi = tc_sigmoid(v[0][i] + bias[wg * 8 + i]);
                                const float go = tc_sigmoid(v[1][i] + bias[16 + wg * 8 + i]);
                                const float gu = tc_tanh(v[2][i] + bias[32 + wg * 8 + i]);
                                cc = gi * gu;
                                h = go * tc_tanh(cc);
                                v[0][i] = gi; v[1][i] = go; v[2][i] = gu;
                            }
                        }
                        hb[i] = __float2bfloat16_rn(h);
                        hv[i] = __bfloat162float(hb[i]);        // the h every consumer sees is the bf16 value
                        cv[i] = cc;
                    }
                    if (u0 == H) hb[0] = __float2bfloat16_rn(1.f);            // first pad column of the bf16 row: the constant
                    else if (u0 + 4 == H) hb[4] = __float2bfloat16_rn(1.f);   // input (see tc_leaf_rows); H is a multiple of 4
                    *reinterpret_cast<uint4*>(c.arena_bf + (size_t)it.x * Hp + u0) = *reinterpret_cast<const uint4*>(hb);
                    if (zrow) *reinterpret_cast<uint4*>(zrow + u0) = *reinterpret_cast<const uint4*>(hb);
                    float* st = c.arena + (size_t)it.x * S;
#pragma unroll
                    for (int i = 0; i < 8; i += 4)
                        if (u0 + i < H) {
                            *reinterpret_cast<float4*>(st + u0 + i) = make_float4(hv[i], hv[i + 1], hv[i + 2], hv[i + 3]);
                            *reinterpret_cast<float4*>(st + H + u0 + i) = make_float4(cv[i], cv[i + 1], cv[i + 2], cv[i + 3]);
                            if (c.gates) {
                                float* gt = c.gates + (size_t)it.x * c.G;
#pragma unroll
                                for (int g = 0; g < NG; ++g)
                                    *reinterpret_cast<float4*>(gt + g * H + u0 + i) =
                                        make_float4(v[g][i], v[g][i + 1], v[g][i + 2], v[g][i + 3]);
                            }
                        }
                }
            } else {
                // warps 0-3 take the first 16-column groups, warps 4-7 the rest
                const int groups = ns / 16, g_lo = (groups + 1) / 2;
                const int g_begin = warp < 4 ? 0 : g_lo, g_end = warp < 4 ? g_lo : groups;
                if (MODE == TC_RNN_FWD) {
                    // all of this thread's accumulator groups in flight, one wait; 32-byte stores
                    constexpr int MAXG = (TC_HP_MAX / 4 / 16 + 1) / 2;
                    uint32_t raw[MAXG][16];
                    // (groups past the slice read unused columns of the 128-column accumulator buffer: never looked at)
#pragma unroll
                    for (int q = 0; q < MAXG; ++q) tc_ld16_issue(lane_base + (uint32_t)((g_begin + q) * 16), raw[q]);
                    tc_wait_ld();
#pragma unroll
                    for (int q = 0; q < MAXG; ++q) {
                        const int gi = g_begin + q;
                        if (gi >= g_end || !live) continue;
                        const int col = slice * ns + gi * 16;                   // column of the padded N range
                        // the state lives in bf16 only: every consumer reads the rounded value
                        __align__(16) __nv_bfloat16 hb[16];
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            float h = 0.f;
                            if (col + i < H) h = tc_tanh(__uint_as_float(raw[q][i]) + sh.ep[gi * 16 + i]);
                            hb[i] = __float2bfloat16_rn(h);
                        }
#pragma unroll
                        for (int i = 0; i < 16; i += 4)                         // first pad column: the constant 1 (H is a multiple of 4)
                            if (col + i == H) hb[i] = __float2bfloat16_rn(1.f);
                        const uint4 lo = *reinterpret_cast<const uint4*>(&hb[0]), hi = *reinterpret_cast<const uint4*>(&hb[8]);
                        st_global_32(c.arena_bf + (size_t)it.x * Hp + col, lo, hi);
                        if (zrow) st_global_32(zrow + col, lo, hi);
                    }
                }
                for (int gi = g_begin; gi < g_end && MODE != TC_RNN_FWD; ++gi) {
                    float v[16];
                    tc_ld16(lane_base + (uint32_t)(gi * 16), v);
                    if (!live) continue;
                    const int col = slice * ns + gi * 16;                       // column of the padded N range
                    if (MODE == TC_LSTM_DE) {
                        // embedding gradient: row tok of dE gathers the contribution of this leaf
#pragma unroll
                        for (int i = 0; i < 16; ++i)
                            if (col + i < c.D) {
                                if (c.dE_fix) fix_add(&c.dE_fix[(size_t)it.y * c.D + col + i], to_fix(v[i]));
                                else atomicAdd(&c.dE[(size_t)it.y * c.D + col + i], v[i]);
                            }
                    } else {
                        // operand gradients: columns [0, Hp) belong to the left callee frame, [Hp, 2Hp) to the right
                        const uint32_t child = col < Hp ? it.y : it.z;
                        const int cc = col < Hp ? col : col - Hp;
                        float* dst = c.dhp + (size_t)child * S + cc;
#pragma unroll
                        for (int i = 0; i < 16; i += 4)
                            if (cc + i < H) *reinterpret_cast<float4*>(dst + i) = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
                    }
                }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            mbar_arrive(acc_empty0 + 8 * b);                   // buffer and records may be reused
        }
    }
    // (writer side of the same ordering: the rows stored above are read by tile copies after the next grid barrier)
    if (WRITES_TILE_ROWS) asm volatile("fence.proxy.async;" ::: "memory");
    tc.g += (uint32_t)(my_tiles * n_chunks);
    tc.T += (uint32_t)my_tiles;
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}

// Leaves in bf16 mode: state(slot) = bf16(E[tok]), pad columns of the row zero.  Each warp takes four
// leaves at a time, so that four rows are in flight per warp.
// bf16 state rows (and, for the TreeLSTM, the bf16 embedding rows) carry the constant 1 in their first pad column
// (column H, when H < Hp): the packed weights have zero rows there, so no contraction of the forward or the gradient
// pass sees it, and the weight-gradient contraction dz (x) [h_l ; h_r] yields the bias gradient sum_t dz_t as its
// column H.
static __device__ void tc_leaf_rows(const DevCtx& c, uint32_t n_items) {
    const int H = c.H, Hp = c.Hp;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) / 32, lane = threadIdx.x % 32;
    const int n_warps = gridDim.x * blockDim.x / 32;
    for (uint32_t i0 = warp * 4; i0 < n_items; i0 += n_warps * 4) {
        uint2 it[4];
        __nv_bfloat16* zrow[4];                               // the half of the caller's operand row that this leaf feeds
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            it[q] = i0 + q < n_items ? __ldcg(reinterpret_cast<const uint2*>(&c.leaf_items[i0 + q])) : make_uint2(0u, 0u);   // {slot, tok}
            const uint32_t zd = i0 + q < n_items ? __ldg(&c.zdst[it[q].x]) : NO_ZDST;
            zrow[q] = zd != NO_ZDST ? c.z_bf + (size_t)(zd >> 1) * 2 * Hp + (size_t)(zd & 1u) * Hp : nullptr;
        }
        for (int k = lane * 8; k < Hp; k += 256) {             // 8 elements per lane: 32 bytes in, 16 bytes out
            float4 v[4][2];
#pragma unroll
            for (int q = 0; q < 4; ++q)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    v[q][e] = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (i0 + q < n_items && k + 4 * e < H)
                        v[q][e] = __ldg(reinterpret_cast<const float4*>(c.E + (size_t)it[q].y * c.D + k + 4 * e));
                }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                if (i0 + q >= n_items) continue;
                __align__(16) __nv_bfloat162 hb[4];
                hb[0] = __floats2bfloat162_rn(v[q][0].x, v[q][0].y); hb[1] = __floats2bfloat162_rn(v[q][0].z, v[q][0].w);
                hb[2] = __floats2bfloat162_rn(v[q][1].x, v[q][1].y); hb[3] = __floats2bfloat162_rn(v[q][1].z, v[q][1].w);
                if (k == H) hb[0].x = __float2bfloat16_rn(1.f);            // the constant input (H is a multiple of 4;
                else if (k + 4 == H) hb[2].x = __float2bfloat16_rn(1.f);   //  k < Hp, so this is a pad column)
                *reinterpret_cast<uint4*>(c.arena_bf + (size_t)it[q].x * Hp + k) = *reinterpret_cast<const uint4*>(hb);
                if (zrow[q]) *reinterpret_cast<uint4*>(zrow[q] + k) = *reinterpret_cast<const uint4*>(hb);
            }
        }
    }
}

// Packed weights (bf16), K halves padded to Hp:
//   Wp [j][k']  (Hp x 2Hp): forward operand,  Wp[j][half*Hp + kk]  = W[j][half*H + kk]
//   WTp[c'][j]  (2Hp x Hp): gradient operand, WTp[half*Hp + kk][j] = W[j][half*H + kk]
static __global__ void __launch_bounds__(256) rdf_pack_w_kernel(const DevCtx c) {
    const int Hp = c.Hp, Kp = 2 * c.Hp, H = c.H;
    for (int idx = blockIdx.x * blockDim.x + threadIdx.x; idx < Hp * Kp; idx += gridDim.x * blockDim.x) {
        const int j = idx / Kp, kp = idx % Kp;
        const int half = kp >= Hp, kk = kp - half * Hp;
        float v = 0.f;
        if (j < H && kk < H) v = c.W[(size_t)j * 2 * H + half * H + kk];
        const __nv_bfloat16 b = __float2bfloat16_rn(v);
        c.Wp[idx] = b;
        c.WTp[(size_t)kp * Hp + j] = b;
    }
}

// TreeLSTM packings (bf16).  Slice-major row order puts everything one block needs in consecutive rows:
//   W5p [(ub*5 + g)*16 + i][k']  (5Hp x 2Hp): gate g of hidden unit u = ub*16 + i, K halves padded to Hp
//   Wxp [(ub*3 + g)*16 + i][k]   (3Hp x Hp) : leaf projection, gates (i, o, u)
//   WT5p[half*Hp + cc][g*Hp + j] (2Hp x 5Hp): gradient operand, = W[g*H + j][half*H + cc]
static __global__ void __launch_bounds__(256) rdf_pack_lstm_kernel(const DevCtx c) {
    const int Hp = c.Hp, Kp = 2 * c.Hp, H = c.H, D = c.D;
    const int stride = gridDim.x * blockDim.x, tid = blockIdx.x * blockDim.x + threadIdx.x;
    for (int idx = tid; idx < 5 * Hp * Kp; idx += stride) {
        const int R = idx / Kp, kp = idx % Kp;
        const int ub = R / 80, g = (R % 80) / 16, u = ub * 16 + R % 16;
        const int half = kp >= Hp, kk = kp - half * Hp;
        float v = 0.f;
        if (u < H && kk < H) v = c.W[(size_t)(g * H + u) * 2 * H + half * H + kk];
        const __nv_bfloat16 b = __float2bfloat16_rn(v);
        c.Wp[idx] = b;
        c.WTp[(size_t)kp * 5 * Hp + g * Hp + u] = b;
    }
    for (int idx = tid; idx < 3 * Hp * Hp; idx += stride) {
        const int R = idx / Hp, k = idx % Hp;
        const int ub = R / 48, g = (R % 48) / 16, u = ub * 16 + R % 16;
        float v = 0.f;
        if (u < H && k < D) v = c.W_x[(size_t)(g * H + u) * D + k];
        const __nv_bfloat16 b = __float2bfloat16_rn(v);
        c.Wxp[idx] = b;
        if (k < Hp) c.WxTp[(size_t)k * 3 * Hp + g * Hp + u] = b;       // WxTp[d][g*Hp + j] = W_x[g*H + j][d]
    }
}

// dE of the TreeLSTM on tensor cores: one launch after the gradient waves, blocks = (row group, 64-column slice of D)
static __global__ void __launch_bounds__(TC_THREADS, 1) rdf_de_tc_kernel(const DevCtx c) {
    extern __shared__ unsigned char dyn_smem[];
    __shared__ TcShared sh;
    if (c.ctl->status != 0) return;                    // an earlier kernel of this call failed
    TcState tc;
    tc_setup(tc, sh, dyn_smem, c.Hp / 64, c.WxTp, 3 * c.Hp, 64);
    tc_pipe<TC_LSTM_DE, 5>(c, tc, sh, 0, c.ctl->all_leaves);
    tc_teardown(tc);
}

// E_bf[v][k] (V x Hp): the embedding table in bf16 with zero pad columns (operand rows of the leaf projection)
static __global__ void __launch_bounds__(256) rdf_pack_e_kernel(const DevCtx c) {
    const size_t total = (size_t)c.V * c.Hp;
    for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (size_t)gridDim.x * blockDim.x) {
        const size_t v = idx / c.Hp;
        const int k = (int)(idx % c.Hp);
        // (first pad column: the constant 1, so that the leaf weight-gradient contraction also yields the leaf bias gradient)
        c.E_bf[idx] = __float2bfloat16_rn(k < c.D ? c.E[v * c.D + k] : k == c.D ? 1.f : 0.f);
    }
}
