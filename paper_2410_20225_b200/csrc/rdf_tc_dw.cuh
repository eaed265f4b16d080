// Weight gradient of the cells on tensor cores:
//     dW[j][k] = sum over cells t of dz_t[j] * x_t[k],      x_t = [h(l_t) ; h(r_t)]
// The contraction runs over the cells, and both operands are stored with the
// contracted index outermost (dz_bf[t][j], arena_bf[.][k]): the "MN-major"
// operand form.  A stage holds 64 cells: for each operand four 64-wide groups
// of j (of k), each as 8 atoms of (8 cells x 128 bytes) with the 128-byte
// swizzle.  Each thread block owns one 256 x 256 tile of dW (two 128-row
// accumulators: all 512 columns of tensor memory) and every splits-th stage
// of the cell list (split-K); partial tiles are added to dW with vector
// atomics, or (reproducible mode) left in a buffer per block and added up in
// split order by a second kernel.  The large tile is what keeps the gather small: an operand row is
// fetched once per tile that needs it, and the gather (16-byte cp.async
// pieces) is what bounds the kernel.  bf16 TreeRNN: the dz rows are stored in
// list order, so that operand arrives as 2D tile copies instead, and column H
// of the product (the constant 1 of the state rows) is the bias gradient.
#pragma once
#include "rdf_tc.cuh"

static const int DW_KT = 64;                          // cells per stage
static const int DW_TILE = 256;                       // rows and columns of dW per block
static const int DW_HALF = DW_KT * DW_TILE * 2;       // 32 KB: one operand of a stage
static const int DW_STAGE = 2 * DW_HALF;
static const int DW_STAGES = 3;
static const int DW_SMEM_BYTES = 1024 + DW_STAGES * DW_STAGE;
static const int DW_PRODUCERS = 128;                  // warps 0-3 gather, warp 4 issues the MMAs, all 8 warps write out

// MN-major operand descriptor: atoms of 64 elements (128 bytes) along M/N by 8 along K;
// lbo = byte distance between atoms along M/N, sbo = between atoms along K.
__device__ __forceinline__ uint64_t tc_desc_mn(uint32_t smem_addr, uint32_t lbo, uint32_t sbo) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)((lbo >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

// What to contract:  out[row(m)][col(n)] += sum over the listed invocations t of A_t[m] * B_t[n]
//   A_t = A + t * lda, Mp padded rows in blocks of Hp (block g, unit j -> output row g * H + j, j < H)
//   mode 0: B_t = [h(l_t) ; h(r_t)] from arena_bf (Np = 2 Hp; column half * Hp + k -> output column half * H + k)
//   mode 1: B_t = E_bf[tok_t]                     (Np = Hp;  column k -> output column k, k < D)
struct DwArgs {
    const uint4* ops;            // {frame, left / token, right, valid} per listed invocation
    const uint32_t* count;
    const __nv_bfloat16* A;
    int lda, Mp, Np, mode;
    float* out;
    int ldo;
    int tiles_n, n_tiles;
    int splits;                  // blocks per tile: block `split` takes the stages split, split + splits, ... of the list
    float* bias_out;             // mode 0 with H < Hp: column H of the left half of B is the constant 1 of the state rows,
                                 // so that column of the product is sum_t A_t = the bias gradient (null: not wanted)
    int a_tiles;                 // 1: the rows of A are in list order (row = position in the list) and are read as 2D tiles
                                 //    through DevCtx::tmap_dz64; the rows after the last listed one are zero up to a multiple of 64
    int b_tiles;                 // 1 (mode 0): B_t is row t of the operand rows z_bf (list order too), read through DevCtx::tmap_z64
    float* partial;              // reproducible mode: [n_tiles * splits][256][256], the block's partial tile (block = split *
                                 // n_tiles + tile) instead of atomics on `out`; null otherwise
};

__global__ void __launch_bounds__(256, 1) rdf_dw_tc_kernel(const __grid_constant__ DevCtx c, const DwArgs a) {
    const uint32_t lbo = 8192u, sbo = 1024u;       // next atom along M/N, next atom along K
    extern __shared__ unsigned char dyn_smem[];
    __shared__ uint32_t tmem_slot;
    __shared__ __align__(8) uint64_t full[DW_STAGES], empty[DW_STAGES], done;
    __shared__ uint4 s_ops[2][DW_KT];                              // records of the stage being copied / the next one
    __shared__ int s_abort;                                        // a producer's bounded wait expired: all producers leave together
    if (c.ctl->status != 0) return;                                // an earlier kernel of this call failed: nothing to contract
    const uint32_t n_cells = *a.count;
    const int tile = blockIdx.x % a.n_tiles, split = blockIdx.x / a.n_tiles;
    // Stages of 64 listed invocations are dealt out round robin, so that at any time the blocks together read one
    // window of consecutive rows (a contiguous range per block reads its rows measurably slower).
    const uint32_t n_stages = (n_cells + DW_KT - 1) / DW_KT;
    if ((uint32_t)split >= n_stages) return;                       // the whole block leaves before any set-up
    const uint32_t n_chunks = (n_stages - (uint32_t)split + (uint32_t)a.splits - 1) / (uint32_t)a.splits;
    const uint32_t t_end = n_cells;
    const int H = c.H, Hp = c.Hp;
    const int m0 = (tile / a.tiles_n) * DW_TILE, n0 = (tile % a.tiles_n) * DW_TILE;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    const uint32_t raw = smem_u32(dyn_smem);
    const uint32_t stage0 = (raw + 1023u) & ~1023u;
    const uint32_t full0 = smem_u32(full), empty0 = smem_u32(empty), done0 = smem_u32(&done);
    if (threadIdx.x == 0) {
        for (int s = 0; s < DW_STAGES; ++s) {
            mbar_init(full0 + 8 * s, DW_PRODUCERS);
            mbar_init(empty0 + 8 * s, 1);
        }
        mbar_init(done0, 1);
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (threadIdx.x < 32) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(&tmem_slot)) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(&tmem_slot);
    bool ok = true;
    if (warp < 4) {
        // ---- producers: a thread copies one 16-byte piece (q) of sixteen cells (tr0 + 4 i) of both operands per stage
        const int q = threadIdx.x & 31, tr0 = threadIdx.x >> 5, atom = q >> 3, c16 = q & 7;
        const int m = m0 + atom * 64 + c16 * 8, n = n0 + atom * 64 + c16 * 8;
        const bool m_in = m < a.Mp, n_in = n < a.Np;
        const __nv_bfloat16* Brows = a.mode == 0 ? c.arena_bf : c.E_bf;
        auto load_op = [&](uint32_t kc) {                          // the record of cell threadIdx.x of stage kc
            const uint32_t idx = ((uint32_t)split + kc * (uint32_t)a.splits) * DW_KT + threadIdx.x;
            return threadIdx.x < DW_KT && kc < n_chunks && idx < t_end ? a.ops[idx] : make_uint4(0u, 0u, 0u, 0u);
        };
        if (threadIdx.x < DW_KT) s_ops[0][threadIdx.x] = load_op(0);
        uint4 op_next = load_op(1);
        asm volatile("bar.sync 1, 128;" ::: "memory");             // the producer warps only
        for (uint32_t kc = 0; kc < n_chunks; ++kc) {
            const uint32_t s = kc % DW_STAGES;
            if (kc >= (uint32_t)DW_STAGES) ok = mbar_wait(c, empty0 + 8 * s, ((kc / DW_STAGES) - 1) & 1u);
            if (!ok) s_abort = 1;
            const uint32_t a_st = stage0 + s * DW_STAGE, b_st = a_st + DW_HALF;
#pragma unroll 4
            for (int i = 0; ok && i < DW_KT / 4; ++i) {
                const int tr = tr0 + 4 * i;
                const uint4 it = s_ops[kc & 1][tr];
                const uint32_t off = atom * 8192 + (tr >> 3) * 1024 + (tr & 7) * 128 + ((c16 ^ (tr & 7)) << 4);
                if (!a.a_tiles) {
                    const bool mv = it.w != 0u && m_in;
                    cp_async16(a_st + off, a.A + (size_t)it.x * a.lda + (mv ? m : 0), mv);
                }
                if (!a.b_tiles) {
                    const bool nv = it.w != 0u && n_in;
                    size_t src = 0;
                    if (nv) src = a.mode == 0 ? (n < Hp ? (size_t)it.y * Hp + n : (size_t)it.z * Hp + (n - Hp)) : (size_t)it.y * Hp + n;
                    cp_async16(b_st + off, Brows + src, nv);
                }
            }
            if (ok && (a.a_tiles || a.b_tiles) && threadIdx.x == 0) {
                // four boxes of 64 rows x 64 columns per operand, each written as the eight swizzled atoms of its column group
                int boxes = 0;
                for (int g = 0; g < 4; ++g) boxes += (a.a_tiles && m0 + g * 64 < a.Mp) + (a.b_tiles && n0 + g * 64 < a.Np);
                mbar_expect_tx(full0 + 8 * s, (uint32_t)boxes * 8192u);
                const int row0 = (int)(((uint32_t)split + kc * (uint32_t)a.splits) * DW_KT);
                for (int g = 0; g < 4; ++g) {
                    if (a.a_tiles && m0 + g * 64 < a.Mp) tma_load_2d(a_st + g * 8192, &c.tmap_dz64, m0 + g * 64, row0, full0 + 8 * s);
                    if (a.b_tiles && n0 + g * 64 < a.Np) tma_load_2d(b_st + g * 8192, &c.tmap_z64, n0 + g * 64, row0, full0 + 8 * s);
                }
            }
            if (ok) cp_async_arrive(full0 + 8 * s);            // arrives when this thread's copies of the stage have landed
            if (threadIdx.x < DW_KT) s_ops[(kc + 1) & 1][threadIdx.x] = op_next;
            op_next = load_op(kc + 2);                         // in flight during the next stage
            asm volatile("bar.sync 1, 128;" ::: "memory");
            if (*reinterpret_cast<volatile int*>(&s_abort)) break;   // the same answer for all producers
        }
    } else if (warp == 4) {
        // ---- MMA issuer: two 128-row accumulators of 256 columns
        if (lane == 0) {
            const uint32_t idesc = tc_idesc(DW_TILE) | (1u << 15) | (1u << 16);    // both operands MN-major
            for (uint32_t kc = 0; kc < n_chunks && ok; ++kc) {
                const uint32_t s = kc % DW_STAGES;
                ok = mbar_wait(c, full0 + 8 * s, (kc / DW_STAGES) & 1u);
                if (!ok) break;
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // cp.async writes -> MMA reads
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t a_st = stage0 + s * DW_STAGE, b_st = a_st + DW_HALF;
#pragma unroll
                for (int ks = 0; ks < DW_KT / 16; ++ks)          // 16 invocations = two K atoms = 2048 bytes per step
#pragma unroll
                    for (int h = 0; h < 2; ++h)
                        tc_mma(tmem + h * DW_TILE, tc_desc_mn(a_st + h * 16384 + ks * 2048, lbo, sbo),
                               tc_desc_mn(b_st + ks * 2048, lbo, sbo), idesc, (kc > 0 || ks > 0) ? 1u : 0u);
                tc_commit(empty0 + 8 * s);
            }
            if (ok) tc_commit(done0);
        }
        __syncwarp();
    }
    // ---- everybody: the accumulators are complete when the last commit has arrived
    ok = mbar_wait(c, done0, 0u);
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (ok && a.partial) {
        float* mine = a.partial + (size_t)blockIdx.x * (DW_TILE * DW_TILE);
        for (int h = 0; h < 2; ++h) {
            const int r = h * 128 + (warp & 3) * 32 + lane;                // row of the tile
            for (int gi = 0; gi < 8; ++gi) {
                float v[16];
                const int cl = (warp >> 2) * 128 + gi * 16;
                tc_ld16(tmem + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)(h * DW_TILE + cl), v);
                float4* dst = reinterpret_cast<float4*>(mine + (size_t)r * DW_TILE + cl);
#pragma unroll
                for (int i = 0; i < 4; ++i) dst[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
            }
        }
    } else if (ok) {
        const int n_limit = a.mode == 0 ? H : c.D;
        for (int h = 0; h < 2; ++h) {
            const int m = m0 + h * 128 + (warp & 3) * 32 + lane;
            const int mj = m % Hp, row = (m / Hp) * H + mj;          // gate block, unit
            for (int gi = 0; gi < 8; ++gi) {
                float v[16];
                const int cl = (warp >> 2) * 128 + gi * 16;
                tc_ld16(tmem + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)(h * DW_TILE + cl), v);
                if (m >= a.Mp || mj >= H || n0 + cl >= a.Np) continue;
                // four columns per atomic: H, D and the row stride of the output are multiples of 4
#pragma unroll
                for (int i = 0; i < 16; i += 4) {
                    const int n = n0 + cl + i;
                    const int k = n < Hp ? n : n - Hp;
                    if (n < a.Np && k < n_limit)
                        atomicAdd(reinterpret_cast<float4*>(&a.out[(size_t)row * a.ldo + (n < Hp ? k : H + k)]),
                                  make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]));
                    else if (a.bias_out && n == H) atomicAdd(&a.bias_out[row], v[i]);
                }
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (threadIdx.x < 32) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
}

// Reproducible mode: out = the partial tiles of every split added up in split order (the blocks that had no stage wrote
// nothing and are not read); rows and columns of the padded tile go to their places in the gradient, column H of the
// left half to the bias gradient.  One thread per four columns of a tile row.
__global__ void __launch_bounds__(256) rdf_dw_reduce_kernel(const __grid_constant__ DevCtx c, const DwArgs a) {
    if (c.ctl->status != 0) return;
    const uint32_t n_stages = (*a.count + DW_KT - 1) / DW_KT;
    const int splits = (int)min((uint32_t)a.splits, n_stages);
    const int H = c.H, Hp = c.Hp, n_limit = a.mode == 0 ? H : c.D;
    const int per_tile = DW_TILE * DW_TILE / 4;
    for (int q = blockIdx.x * blockDim.x + threadIdx.x; q < a.n_tiles * per_tile; q += gridDim.x * blockDim.x) {
        const int tile = q / per_tile, e = q % per_tile, r = e / (DW_TILE / 4), c4 = (e % (DW_TILE / 4)) * 4;
        const int m = (tile / a.tiles_n) * DW_TILE + r, n = (tile % a.tiles_n) * DW_TILE + c4;
        const int mj = m % Hp, row = (m / Hp) * H + mj;              // gate block, unit
        if (m >= a.Mp || mj >= H || n >= a.Np) continue;
        const int k = n < Hp ? n : n - Hp;
        const bool bias = a.bias_out && n == H;
        if (k >= n_limit && !bias) continue;
        float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int sp = 0; sp < splits; ++sp) {
            const float4 v = *reinterpret_cast<const float4*>(a.partial + ((size_t)sp * a.n_tiles + tile) * (DW_TILE * DW_TILE) + (size_t)r * DW_TILE + c4);
            t.x += v.x; t.y += v.y; t.z += v.z; t.w += v.w;
        }
        if (k < n_limit) *reinterpret_cast<float4*>(&a.out[(size_t)row * a.ldo + (n < Hp ? k : H + k)]) = t;
        else a.bias_out[row] = t.x;
    }
}
