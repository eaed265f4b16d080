// Tensor-core path (sm_100a: tcgen05 + tensor memory) for the dense cell
// contraction of the bf16 workloads:
//     D[128 cells x Np] = A[128 x Kp] * Wp[Np x Kp]^T,   fp32 accumulation in TMEM
// A rows are the gathered operand states [h_l ; h_r] of the ready cells, in
// bf16; Wp is the weight matrix packed to bf16 with each half of K padded to a
// multiple of 64.  Both operands are K-major; they are staged by all threads
// into shared memory in the 128-byte-swizzled layout the MMA reads (8-row
// groups of 1024 bytes, 16-byte chunks XOR-ed with the row index), one elected
// thread issues the MMAs, completion is signalled on an mbarrier by
// tcgen05.commit, and the epilogue reads the accumulators back with
// tcgen05.ld.  Every wait is bounded; on expiry the status word is set.
#pragma once
#include <cuda_bf16.h>

#include "rdf_exec.h"

static const int TC_M = 128;          // cells per tile (TMEM lanes)
static const int TC_KC = 64;          // bf16 elements per staged K chunk = one 128-byte swizzled row
static const int TC_NMAX = 320;       // widest packed N (TMEM columns used)
static const int TC_STAGE_A = TC_M * 128;
static const int TC_STAGE_B = TC_NMAX * 128;
static const int TC_STAGE = TC_STAGE_A + TC_STAGE_B;            // 57344 bytes, a multiple of 1024
static const int TC_SMEM_BYTES = 2 * TC_STAGE + 1024;           // two stages + slack to align to 1024

struct TcState {
    uint32_t tmem_base;      // TMEM address returned by tcgen05.alloc
    uint32_t stage_addr;     // shared-space address of stage 0 (1024-byte aligned)
    uint32_t mbar_addr;      // shared-space address of the two mbarriers
    uint32_t iter;           // K chunks issued so far (stage = iter & 1)
    unsigned char* stage_ptr;
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

// One-time set-up per kernel (all threads call it): TMEM allocation by warp 0, mbarriers.
__device__ __forceinline__ void tc_setup(TcState& tc, unsigned char* dyn_smem, uint32_t* tmem_slot, uint64_t* mbars) {
    const uint32_t raw = smem_u32(dyn_smem);
    const uint32_t aligned = (raw + 1023u) & ~1023u;
    tc.stage_addr = aligned;
    tc.stage_ptr = dyn_smem + (aligned - raw);
    tc.mbar_addr = smem_u32(mbars);
    tc.iter = 0;
    if (threadIdx.x == 0) {
        mbar_init(tc.mbar_addr, 1);
        mbar_init(tc.mbar_addr + 8, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (threadIdx.x < 32) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(tmem_slot)) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    tc.tmem_base = *reinterpret_cast<volatile uint32_t*>(tmem_slot);
}

__device__ __forceinline__ void tc_teardown(const TcState& tc) {
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (threadIdx.x < 32)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tc.tmem_base) : "memory");
}

// byte offset of 16-byte chunk c16 of row r inside a swizzled [rows x 128 bytes] operand tile
__device__ __forceinline__ uint32_t swz(int r, int c16) {
    return (uint32_t)((r >> 3) * 1024 + (r & 7) * 128 + ((c16 ^ (r & 7)) << 4));
}

// TreeRNN cell on tensor cores: state(out) = tanh(W [state(l); state(r)] + b) for n_items ready cells.
// arena_bf: bf16 states, row stride Hp (a multiple of 64, pad columns zero); Wp: [Np = Hp][Kp = 2 Hp] bf16.
__device__ void tc_rnn_cell_tiles(const DevCtx& c, TcState& tc, uint32_t n_items) {
    const int H = c.H, Hp = c.Hp, Kp = 2 * c.Hp, Np = c.Hp;
    const int n_chunks = Kp / TC_KC, n_half = Np / 2;            // two MMAs of N = Np / 2 per K step
    const uint32_t idesc = tc_idesc(n_half);
    const int tiles = (n_items + TC_M - 1) / TC_M;
    const __nv_bfloat16* arena_bf = c.arena_bf;
    bool ok = true;
    for (int tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x) {
        const int row0 = tile * TC_M;
        for (int kc = 0; kc < n_chunks && ok; ++kc) {
            const uint32_t s = tc.iter & 1u;
            // the MMAs that last read this stage must have completed
            if (tc.iter >= 2) ok = mbar_wait(c, tc.mbar_addr + 8 * s, ((tc.iter >> 1) - 1) & 1u);
            unsigned char* sa = tc.stage_ptr + s * TC_STAGE;
            unsigned char* sb = sa + TC_STAGE_A;
            // A chunk: 128 rows x 8 chunks of 16 bytes, gathered from the operand states
            const int koff = kc * TC_KC;
            for (int p = threadIdx.x; p < TC_M * 8; p += blockDim.x) {
                const int r = p >> 3, c16 = p & 7;
                uint4 v = make_uint4(0u, 0u, 0u, 0u);
                if (row0 + r < (int)n_items) {
                    const uint4 it = __ldcg(reinterpret_cast<const uint4*>(&c.cell_items[row0 + r]));   // {out, l, r, -}
                    const uint32_t src = koff < Hp ? it.y : it.z;
                    const int kk = (koff < Hp ? koff : koff - Hp) + c16 * 8;
                    v = __ldcg(reinterpret_cast<const uint4*>(arena_bf + (size_t)src * Hp + kk));
                }
                *reinterpret_cast<uint4*>(sa + swz(r, c16)) = v;
            }
            // B chunk: Np rows of the packed weights
            for (int p = threadIdx.x; p < Np * 8; p += blockDim.x) {
                const int r = p >> 3, c16 = p & 7;
                const uint4 v = __ldg(reinterpret_cast<const uint4*>(c.Wp + (size_t)r * Kp + koff + c16 * 8));
                *reinterpret_cast<uint4*>(sb + swz(r, c16)) = v;
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // generic-proxy writes -> async proxy reads
            __syncthreads();
            if (threadIdx.x == 0) {
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t a_addr = tc.stage_addr + s * TC_STAGE, b_addr = a_addr + TC_STAGE_A;
#pragma unroll
                for (int ks = 0; ks < TC_KC / 16; ++ks) {
                    const uint32_t acc = (kc > 0 || ks > 0) ? 1u : 0u;
                    const uint64_t ad = tc_desc(a_addr + ks * 32);
                    tc_mma(tc.tmem_base, ad, tc_desc(b_addr + ks * 32), idesc, acc);
                    tc_mma(tc.tmem_base + n_half, ad, tc_desc(b_addr + n_half * 128 + ks * 32), idesc, acc);
                }
                tc_commit(tc.mbar_addr + 8 * s);
            }
            ++tc.iter;
        }
        // accumulators complete when the last commit has arrived
        if (ok) ok = mbar_wait(c, tc.mbar_addr + 8 * ((tc.iter - 1) & 1u), ((tc.iter - 1) >> 1) & 1u);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (ok) {
            // epilogue: warp w reads TMEM lanes 32 (w % 4) ..; warps 0-3 take the low half of the columns, 4-7 the high half
            const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
            const int row = (warp & 3) * 32 + lane;
            const int cbase = (warp >> 2) * n_half;
            const bool live = row0 + row < (int)n_items;
            const uint32_t out = live ? __ldcg(&c.cell_items[row0 + row].out) : 0u;
            for (int cc = 0; cc < n_half; cc += 16) {
                float v[16];
                tc_ld16(tc.tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)(cbase + cc), v);
                if (!live) continue;
                const int col = cbase + cc;
                __align__(16) __nv_bfloat16 hb[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    float h = 0.f;
                    if (col + i < H) h = tanhf(v[i] + __ldg(&c.b[col + i]));
                    hb[i] = __float2bfloat16_rn(h);
                    v[i] = __bfloat162float(hb[i]);          // the state every consumer sees is the bf16 value
                }
                uint4* dstb = reinterpret_cast<uint4*>(c.arena_bf + (size_t)out * Hp + col);
                dstb[0] = *reinterpret_cast<const uint4*>(&hb[0]);
                dstb[1] = *reinterpret_cast<const uint4*>(&hb[8]);
                float* dstf = c.arena + (size_t)out * H + col;
#pragma unroll
                for (int i = 0; i < 16; i += 4)
                    if (col + i < H) *reinterpret_cast<float4*>(dstf + i) = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
            }
        }
        // TMEM and the stages may be overwritten by the next tile only after everybody has read them
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();
    }
}

// Leaves in bf16 mode: state(slot) = E[tok] in both arenas (pad columns of the bf16 row are zero).
__device__ void tc_leaf_rows(const DevCtx& c, uint32_t n_items) {
    const int H = c.H, Hp = c.Hp;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) / 32, lane = threadIdx.x % 32;
    const int n_warps = gridDim.x * blockDim.x / 32;
    for (uint32_t i = warp; i < n_items; i += n_warps) {
        const uint2 it = __ldcg(reinterpret_cast<const uint2*>(&c.leaf_items[i]));          // {slot, tok}
        const float* src = c.E + (size_t)it.y * c.D;
        float* dst = c.arena + (size_t)it.x * H;
        __nv_bfloat16* dstb = c.arena_bf + (size_t)it.x * Hp;
        for (int k = lane; k < Hp; k += 32) {
            const float v = k < H ? __ldg(src + k) : 0.f;
            const __nv_bfloat16 b = __float2bfloat16_rn(v);
            dstb[k] = b;
            if (k < H) dst[k] = __bfloat162float(b);
        }
    }
}

// Wp[j][k'] (bf16): rows j < H are W[j], with the left half of K at k' = k and the right half at k' = Hp + (k - H).
__global__ void __launch_bounds__(256) rdf_pack_w_kernel(const DevCtx c) {
    const int Hp = c.Hp, Kp = 2 * c.Hp, H = c.H;
    for (int idx = blockIdx.x * blockDim.x + threadIdx.x; idx < Hp * Kp; idx += gridDim.x * blockDim.x) {
        const int j = idx / Kp, kp = idx % Kp;
        const int half = kp >= Hp, kk = kp - half * Hp;
        float v = 0.f;
        if (j < H && kk < H) v = c.W[(size_t)j * 2 * H + half * H + kk];
        c.Wp[idx] = __float2bfloat16_rn(v);
    }
}
