// Tensor-core path (sm_100a: tcgen05 + tensor memory) for the dense
// contractions of the bf16 TreeRNN workloads, forward and operand-gradient:
//
//   forward :  D[128 cells x NS] = A[128 x 2Hp] * Wp [NS x 2Hp]^T     A row = [h_l ; h_r] (bf16 states, gathered)
//   backward:  D[128 cells x NS] = A[128 x  Hp] * WTp[NS x  Hp]^T     A row = dz (bf16),  D = slice of [dh_l ; dh_r]
//
// Weight-stationary: the packed weight matrix is split along N into slices of
// NS = Hp / 4 rows; a thread block owns one slice for the whole kernel and
// keeps it in shared memory (loaded once, <= 100 KB), so per tile only the
// gathered operand rows move.  A rows are streamed with cp.async through a
// 4-stage ring of 128-byte-swizzled [128 x 64] bf16 tiles (8-row groups of
// 1024 bytes, 16-byte chunks XOR-ed with the row index: the K-major layout the
// MMA reads); one thread issues the tcgen05.mma instructions, tcgen05.commit
// signals an mbarrier per stage, accumulators live in tensor memory and the
// epilogue reads them back with tcgen05.ld.  Every wait is bounded.
#pragma once
#include <cuda_bf16.h>

#include "rdf_exec.h"

static const int TC_M = 128;                 // cells per tile (TMEM lanes)
static const int TC_KC = 64;                 // bf16 elements per staged K chunk = one 128-byte swizzled row
static const int TC_STAGES = 4;
static const int TC_A_STAGE = TC_M * 128;    // 16 KB
static const int TC_HP_MAX = 320;            // widest padded hidden size the resident slice is sized for
static const int TC_B_MAX = TC_HP_MAX * TC_HP_MAX;                               // (Hp/4) rows x 2Hp x 2 bytes
static const int TC_SMEM_BYTES = 1024 + TC_B_MAX + TC_STAGES * TC_A_STAGE;       // + slack to align to 1024
static const int TC_TMEM_COLS = 128;

struct TcState {
    uint32_t tmem_base;      // TMEM address returned by tcgen05.alloc
    uint32_t b_addr;         // shared-space address of the resident weight slice (1024-byte aligned)
    uint32_t a_addr;         // shared-space address of A stage 0
    uint32_t mbar_addr;      // shared-space address of the per-stage mbarriers
    uint32_t iter;           // K chunks issued so far (stage = iter % TC_STAGES)
    int      ns, n_split, n_chunks;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t addr, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(addr), "r"(count) : "memory");
}

// Bounded wait for the phase with the given parity.  Returns false on expiry.
__device__ __forceinline__ bool mbar_wait(const DevCtx& c, uint32_t addr, uint32_t parity) {
    const long long t0 = clock64();
    for (;;) {
        uint32_t done;
        asm volatile(
            "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
            : "=r"(done) : "r"(addr), "r"(parity) : "memory");
        if (done) return true;
        if (clock64() - t0 > c.spin_limit) {
            set_status(c, RDF_ERR_TIMEOUT);
            return false;
        }
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

// 16-byte asynchronous copy global -> shared through L2; `valid == false` writes zeros
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
    const int n = valid ? 16 : 0;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(n) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// byte offset of 16-byte chunk c16 of row r inside a swizzled [rows x 128 bytes] operand tile
__device__ __forceinline__ uint32_t swz(int r, int c16) {
    return (uint32_t)((r >> 3) * 1024 + (r & 7) * 128 + ((c16 ^ (r & 7)) << 4));
}

// One-time set-up per kernel (all threads call it): TMEM allocation by warp 0, mbarriers, and the
// block's resident slice of the packed weights: rows [slice * ns, +ns) of Bp[. x Kp], chunk by chunk.
__device__ __forceinline__ void tc_setup(TcState& tc, unsigned char* dyn_smem, uint32_t* tmem_slot, uint64_t* mbars,
                                         const __nv_bfloat16* Bp, int Kp, int ns, int n_split) {
    const uint32_t raw = smem_u32(dyn_smem);
    const uint32_t aligned = (raw + 1023u) & ~1023u;
    tc.b_addr = aligned;
    tc.a_addr = aligned + TC_B_MAX;
    tc.mbar_addr = smem_u32(mbars);
    tc.iter = 0;
    tc.ns = ns;
    tc.n_split = n_split;
    tc.n_chunks = Kp / TC_KC;
    if (threadIdx.x == 0) {
        for (int s = 0; s < TC_STAGES; ++s) mbar_init(tc.mbar_addr + 8 * s, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (threadIdx.x < 32) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "n"(TC_TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    const int slice = blockIdx.x % n_split;
    unsigned char* bp = dyn_smem + (aligned - raw);
    const int chunk_bytes = ns * 128;
    for (int p = threadIdx.x; p < tc.n_chunks * ns * 8; p += blockDim.x) {
        const int kc = p / (ns * 8), q = p % (ns * 8), r = q >> 3, c16 = q & 7;
        const uint4 v = *reinterpret_cast<const uint4*>(Bp + (size_t)(slice * ns + r) * Kp + kc * TC_KC + c16 * 8);
        *reinterpret_cast<uint4*>(bp + kc * chunk_bytes + swz(r, c16)) = v;
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    tc.tmem_base = *reinterpret_cast<volatile uint32_t*>(tmem_slot);
}

__device__ __forceinline__ void tc_teardown(const TcState& tc) {
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (threadIdx.x < 32)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tc.tmem_base), "n"(TC_TMEM_COLS) : "memory");
}

// One 128-cell tile loop.  FWD = true : cells cell_items[0, n_items); A row = [state(l) ; state(r)] in bf16;
//                                         epilogue state(out) = tanh(D + b) into both arenas.
//                          FWD = false: cells all_cells[first, first + n_items); A row = dz in bf16;
//                                         epilogue writes D into the incoming-gradient rows of the operand frames.
// s_items: 128 x uint4 of shared memory for the tile's cell records.
template <bool FWD>
__device__ void tc_tiles(const DevCtx& c, TcState& tc, uint4* s_items, uint32_t first, uint32_t n_items) {
    const int H = c.H, Hp = c.Hp, ns = tc.ns, n_chunks = tc.n_chunks;
    const int slice = blockIdx.x % tc.n_split, rg = blockIdx.x / tc.n_split, n_rg = gridDim.x / tc.n_split;
    if (rg >= n_rg) return;                                    // blocks beyond the last full group sit this out
    const uint32_t idesc = tc_idesc(ns);
    const int tiles = (n_items + TC_M - 1) / TC_M;
    const __nv_bfloat16* Arows = FWD ? c.arena_bf : c.dz_bf;
    bool ok = true;
    for (int tile = rg; tile < tiles && ok; tile += n_rg) {
        const int row0 = tile * TC_M;
        if (threadIdx.x < TC_M) {
            uint4 it = make_uint4(0u, 0u, 0u, 0u);
            const int row = row0 + threadIdx.x;
            if (row < (int)n_items) {
                if (FWD) {
                    it = __ldcg(reinterpret_cast<const uint4*>(&c.cell_items[row]));   // {out, l, r, -}
                } else {
                    const uint32_t t = __ldcg(&c.all_cells[first + row]);
                    it.x = t; it.y = __ldcg(&c.op_l[t]); it.z = __ldcg(&c.op_r[t]);
                }
                it.w = 1u;
            }
            s_items[threadIdx.x] = it;
        }
        __syncthreads();
        const uint32_t it0 = tc.iter;
        auto issue = [&](int kc) {
            const uint32_t g = it0 + kc, s = g % TC_STAGES;
            // the MMAs that last read this stage must have completed
            if (g >= TC_STAGES) ok = mbar_wait(c, tc.mbar_addr + 8 * s, ((g / TC_STAGES) - 1) & 1u) && ok;
            const int koff = kc * TC_KC;
            for (int p = threadIdx.x; p < TC_M * 8; p += blockDim.x) {
                const int r = p >> 3, c16 = p & 7;
                const uint4 it = s_items[r];
                size_t src;
                if (FWD) src = (size_t)(koff < Hp ? it.y : it.z) * Hp + (koff < Hp ? koff : koff - Hp) + c16 * 8;
                else src = (size_t)it.x * Hp + koff + c16 * 8;
                cp_async16(tc.a_addr + s * TC_A_STAGE + swz(r, c16), Arows + src, it.w != 0u);
            }
            cp_async_commit();
        };
        issue(0);
        if (n_chunks > 1) issue(1); else cp_async_commit();
        for (int kc = 0; kc < n_chunks; ++kc) {
            if (kc + 2 < n_chunks) issue(kc + 2); else cp_async_commit();
            cp_async_wait<2>();                                          // this thread's copies of chunk kc have landed
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy writes -> async-proxy reads
            __syncthreads();
            if (threadIdx.x == 0) {
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t s = (it0 + kc) % TC_STAGES;
                const uint32_t a = tc.a_addr + s * TC_A_STAGE, b = tc.b_addr + kc * ns * 128;
#pragma unroll
                for (int ks = 0; ks < TC_KC / 16; ++ks)
                    tc_mma(tc.tmem_base, tc_desc(a + ks * 32), tc_desc(b + ks * 32), idesc, (kc > 0 || ks > 0) ? 1u : 0u);
                tc_commit(tc.mbar_addr + 8 * s);
            }
        }
        tc.iter = it0 + n_chunks;
        // accumulators are complete when the last commit has arrived
        {
            const uint32_t g = tc.iter - 1;
            if (ok) ok = mbar_wait(c, tc.mbar_addr + 8 * (g % TC_STAGES), (g / TC_STAGES) & 1u);
        }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (ok) {
            // warp w reads TMEM lanes 32 (w % 4) ..; warps 0-3 take the first 16-column groups, warps 4-7 the rest
            const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
            const int row = (warp & 3) * 32 + lane;
            const int groups = ns / 16, g_lo = (groups + 1) / 2;
            const int g_begin = warp < 4 ? 0 : g_lo, g_end = warp < 4 ? g_lo : groups;
            const uint4 it = s_items[row];
            const bool live = it.w != 0u;
            for (int gi = g_begin; gi < g_end; ++gi) {
                float v[16];
                tc_ld16(tc.tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)(gi * 16), v);
                if (!live) continue;
                const int col = slice * ns + gi * 16;                       // column of the padded N range
                if (FWD) {
                    __align__(16) __nv_bfloat16 hb[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        float h = 0.f;
                        if (col + i < H) h = tanhf(v[i] + __ldg(&c.b[col + i]));
                        hb[i] = __float2bfloat16_rn(h);
                        v[i] = __bfloat162float(hb[i]);      // the state every consumer sees is the bf16 value
                    }
                    uint4* dstb = reinterpret_cast<uint4*>(c.arena_bf + (size_t)it.x * Hp + col);
                    dstb[0] = *reinterpret_cast<const uint4*>(&hb[0]);
                    dstb[1] = *reinterpret_cast<const uint4*>(&hb[8]);
                    float* dstf = c.arena + (size_t)it.x * H + col;
#pragma unroll
                    for (int i = 0; i < 16; i += 4)
                        if (col + i < H) *reinterpret_cast<float4*>(dstf + i) = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
                } else {
                    const uint32_t child = col < Hp ? it.y : it.z;
                    const int cc = col < Hp ? col : col - Hp;
                    float* dst = c.dhp + (size_t)child * H + cc;
#pragma unroll
                    for (int i = 0; i < 16; i += 4)
                        if (cc + i < H) *reinterpret_cast<float4*>(dst + i) = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
                }
            }
        }
        // TMEM, the stages and s_items may be overwritten by the next tile only after everybody has read them
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();
    }
}

// Leaves in bf16 mode: state(slot) = E[tok] in both arenas (pad columns of the bf16 row are zero).
static __device__ void tc_leaf_rows(const DevCtx& c, uint32_t n_items) {
    const int H = c.H, Hp = c.Hp;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) / 32, lane = threadIdx.x % 32;
    const int n_warps = gridDim.x * blockDim.x / 32;
    for (uint32_t i = warp; i < n_items; i += n_warps) {
        const uint2 it = __ldcg(reinterpret_cast<const uint2*>(&c.leaf_items[i]));          // {slot, tok}
        const float* src = c.E + (size_t)it.y * c.D;
        float* dst = c.arena + (size_t)it.x * H;
        __nv_bfloat16* dstb = c.arena_bf + (size_t)it.x * Hp;
        for (int k = lane * 8; k < Hp; k += 256) {             // 8 elements per lane: 32 bytes in, 16 + 32 bytes out
            float v[8];
#pragma unroll
            for (int i = 0; i < 8; i += 4) {
                float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
                if (k + i < H) t = __ldg(reinterpret_cast<const float4*>(src + k + i));
                v[i] = t.x; v[i + 1] = t.y; v[i + 2] = t.z; v[i + 3] = t.w;
            }
            __align__(16) __nv_bfloat16 hb[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                hb[i] = __float2bfloat16_rn(v[i]);
                v[i] = __bfloat162float(hb[i]);
            }
            *reinterpret_cast<uint4*>(dstb + k) = *reinterpret_cast<const uint4*>(hb);
#pragma unroll
            for (int i = 0; i < 8; i += 4)
                if (k + i < H) *reinterpret_cast<float4*>(dst + k + i) = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
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
