// Reverse mode (Section 4).  The forward run retains, per invocation, its
// frame, its state and the operands of the operator that produced the state.
// The gradient pass re-enters every invocation under the tag (frame) that its
// forward Call_i created: wave 0 holds the invocations called from `result`,
// each wave hands the gradients of a cell's operands to the frames of the two
// calls it made (Call_1 / Call_2 replayed through the retained operand frames),
// until the leaves are reached.  Parameter gradients are sums over all
// invocations and are formed after the waves as dense contractions over the
// retained per-invocation values.
#include <algorithm>
#include <cstring>
#include <type_traits>

#include "rdf_exec.h"
#include "rdf_tc.cuh"
#include "rdf_tc_dw.cuh"

static const int MAX_CLASSES = 8;

// ---------------------------------------------------------------- loss head
// Eight hidden units of a state row as floats: from the fp32 arena (row stride S) or, for the bf16
// TreeRNN, from the bf16 arena (row stride Hp, pad columns zero).
__device__ __forceinline__ void unpack_bf8(const uint4& v, float (&x)[8]) {
    const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 f = __bfloat1622float2(p[i]);
        x[2 * i] = f.x; x[2 * i + 1] = f.y;
    }
}

// Loss head and its parameter gradients in one streaming pass over the retained states:
//   per invocation f:  z = W_s h_f + b_s;  loss += logsumexp(z) - z[label];  dlog_f = softmax(z) - onehot
//   dW_s[k][j] = sum_f dlog_f[k] * h_f[j];   db_s[k] = sum_f dlog_f[k]
// A block owns a contiguous range of invocations (consecutive frame ids = consecutive rows) and moves
// it through shared memory in slabs of `fr` rows with bulk asynchronous copies, two slabs in flight.
// BF: rows of the bf16 arena (Hp bf16, pad columns zero); else rows of the fp32 arena (S floats).
static const int LH_MAX_ROWS = 64;          // rows per slab
static const int LH_SLAB_BYTES = 48 * 1024;
static const int GRAD_MAX_H = 1024;         // widest hidden size of the gradient pass

template <bool BF>
__global__ void __launch_bounds__(256) rdf_loss_heads_kernel(const DevCtx c, int fr, int rowbytes) {
    if (c.ctl->status != 0) return;                    // an earlier kernel of this call failed: its lists and rows are not to be trusted
    extern __shared__ __align__(128) unsigned char slab_smem[];
    __shared__ __align__(8) uint64_t mbars[2];
    __shared__ __align__(16) float s_dl[LH_MAX_ROWS][8];
    __shared__ int s_lab[2][LH_MAX_ROWS];
    __shared__ float warp_loss[8];
    const uint32_t F = c.ctl->frame_count.v, B = (uint32_t)c.B;
    const uint32_t n = F > B ? F - B : 0u, per = (n + gridDim.x - 1) / gridDim.x;
    const uint32_t f0 = min(F, B + blockIdx.x * per), f1 = min(F, f0 + per);
    const int n_slabs = (int)((f1 - f0 + fr - 1) / fr);
    const int tid = threadIdx.x, lane = tid % 32, wib = tid / 32;
    const int H = c.H, C = c.n_classes;
    const uint32_t mbar = smem_u32(mbars), stage0 = smem_u32(slab_smem);
    const uint32_t stage_bytes = (uint32_t)fr * rowbytes;
    const unsigned char* rows = BF ? reinterpret_cast<const unsigned char*>(c.arena_bf)
                                   : reinterpret_cast<const unsigned char*>(c.arena);
    if (tid == 0) {
        mbar_init(mbar, 1);
        mbar_init(mbar + 8, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    auto issue = [&](int i) {
        const uint32_t fs = f0 + (uint32_t)i * fr, cnt = min((uint32_t)fr, f1 - fs);
        if (tid == 0) {
            const uint32_t bytes = cnt * rowbytes, mb = mbar + 8 * (i & 1);
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(mb), "r"(bytes) : "memory");
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(stage0 + (i & 1) * stage_bytes), "l"(rows + (size_t)fs * rowbytes), "r"(bytes), "r"(mb) : "memory");
        }
        if (tid < (int)cnt) s_lab[i & 1][tid] = __ldg(&c.label[(int)c.frames[fs + tid].arg]);
    };
    // W_s in shared memory, behind the two slab stages
    float* s_ws = reinterpret_cast<float*>(slab_smem + 2 * (size_t)stage_bytes);
    for (int q = tid; q < C * H; q += 256) s_ws[q] = __ldg(&c.W_s[q]);
    // dW_s: G groups of four hidden units, n_sets threads per group (GRAD_MAX_H / 4 = 256 threads at most per set)
    const int G = (H + 3) / 4, n_sets = 256 / G, cg = tid % G, set = tid / G;
    float acc[4][MAX_CLASSES];
#pragma unroll
    for (int e = 0; e < 4; ++e)
#pragma unroll
        for (int k = 0; k < MAX_CLASSES; ++k) acc[e][k] = 0.f;
    float my_loss = 0.f, my_dbs = 0.f;
    bool ok = true;
    if (n_slabs > 0) issue(0);
    for (int i = 0; i < n_slabs && ok; ++i) {
        if (i + 1 < n_slabs) issue(i + 1);             // its stage was released by the barrier that ended slab i - 1
        const uint32_t fs = f0 + (uint32_t)i * fr, cnt = min((uint32_t)fr, f1 - fs);
        ok = __syncthreads_and(mbar_wait(c, mbar + 8 * (i & 1), (uint32_t)(i >> 1) & 1u)) != 0;
        if (!ok) break;                                // the whole block agrees
        const unsigned char* st = slab_smem + (size_t)(i & 1) * stage_bytes;
        // ---- logits, loss, dlog: a warp takes four rows at a time, a lane 8 hidden units per 256;
        //      a piece of W_s (from shared memory) serves all four rows
        for (uint32_t fb = wib * 4; fb < cnt; fb += 32) {
            float z[4][MAX_CLASSES];
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int k = 0; k < MAX_CLASSES; ++k) z[r][k] = 0.f;
            for (int j = lane * 8; j < H; j += 256) {
                float x[4][8];
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    const unsigned char* row = st + (size_t)min(fb + r, cnt - 1) * rowbytes;
                    if (BF) {
                        unpack_bf8(*reinterpret_cast<const uint4*>(row + 2 * j), x[r]);
                    } else {
                        const float4 a = *reinterpret_cast<const float4*>(row + 4 * j);
                        const float4 b = j + 4 < H ? *reinterpret_cast<const float4*>(row + 4 * j + 16) : make_float4(0.f, 0.f, 0.f, 0.f);
                        x[r][0] = a.x; x[r][1] = a.y; x[r][2] = a.z; x[r][3] = a.w;
                        x[r][4] = b.x; x[r][5] = b.y; x[r][6] = b.z; x[r][7] = b.w;
                    }
                }
#pragma unroll
                for (int k = 0; k < MAX_CLASSES; ++k)
                    if (k < C) {
                        const float4 w0 = *reinterpret_cast<const float4*>(&s_ws[k * H + j]);
                        const float4 w1 = j + 4 < H ? *reinterpret_cast<const float4*>(&s_ws[k * H + j + 4]) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                        for (int r = 0; r < 4; ++r)
                            z[r][k] += w0.x * x[r][0] + w0.y * x[r][1] + w0.z * x[r][2] + w0.w * x[r][3] +
                                       w1.x * x[r][4] + w1.y * x[r][5] + w1.z * x[r][6] + w1.w * x[r][7];
                    }
            }
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int k = 0; k < MAX_CLASSES; ++k)
                    if (k < C)
                        for (int o = 16; o > 0; o >>= 1) z[r][k] += __shfl_xor_sync(0xffffffffu, z[r][k], o);
            // lane r finishes row fb + r
            float zr[MAX_CLASSES];
#pragma unroll
            for (int k = 0; k < MAX_CLASSES; ++k) zr[k] = lane == 0 ? z[0][k] : lane == 1 ? z[1][k] : lane == 2 ? z[2][k] : z[3][k];
            const uint32_t fi = fb + lane;
            if (lane < 4 && fi < cnt) {
                const int lab = s_lab[i & 1][fi];
                float m = -INFINITY;
#pragma unroll
                for (int k = 0; k < MAX_CLASSES; ++k)
                    if (k < C) {
                        zr[k] += __ldg(&c.b_s[k]);
                        m = fmaxf(m, zr[k]);
                    }
                float sum = 0.f, zl = 0.f;
#pragma unroll
                for (int k = 0; k < MAX_CLASSES; ++k)
                    if (k < C) {
                        sum += expf(zr[k] - m);
                        if (k == lab) zl = zr[k];
                    }
                my_loss += logf(sum) + m - zl;
                float d[MAX_CLASSES];
#pragma unroll
                for (int k = 0; k < MAX_CLASSES; ++k) d[k] = k < C ? expf(zr[k] - m) / sum - (k == lab ? 1.f : 0.f) : 0.f;
                const float4 lo = make_float4(d[0], d[1], d[2], d[3]), hi = make_float4(d[4], d[5], d[6], d[7]);
                *reinterpret_cast<float4*>(c.dlog + (size_t)(fs + fi) * 8) = lo;
                *reinterpret_cast<float4*>(c.dlog + (size_t)(fs + fi) * 8 + 4) = hi;
                *reinterpret_cast<float4*>(&s_dl[fi][0]) = lo;
                *reinterpret_cast<float4*>(&s_dl[fi][4]) = hi;
            }
        }
        __syncthreads();
        // ---- dW_s, db_s: a thread owns four hidden units and every n_sets-th row; sums stay in registers
        if (tid < n_sets * G) {
            for (uint32_t fi = set; fi < cnt; fi += n_sets) {
                const unsigned char* row = st + (size_t)fi * rowbytes;
                float hx[4];
                if (BF) {
                    const uint2 v = *reinterpret_cast<const uint2*>(row + 8 * cg);
                    const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&v.x));
                    const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&v.y));
                    hx[0] = a.x; hx[1] = a.y; hx[2] = b.x; hx[3] = b.y;
                } else {
                    const float4 v = *reinterpret_cast<const float4*>(row + 16 * cg);
                    hx[0] = v.x; hx[1] = v.y; hx[2] = v.z; hx[3] = v.w;
                }
                const float4 d0 = *reinterpret_cast<const float4*>(&s_dl[fi][0]);
                const float4 d1 = *reinterpret_cast<const float4*>(&s_dl[fi][4]);
                const float dl[MAX_CLASSES] = {d0.x, d0.y, d0.z, d0.w, d1.x, d1.y, d1.z, d1.w};
#pragma unroll
                for (int e = 0; e < 4; ++e)
#pragma unroll
                    for (int k = 0; k < MAX_CLASSES; ++k) acc[e][k] = fmaf(dl[k], hx[e], acc[e][k]);
            }
        }
        if (tid < C)
            for (uint32_t fi = 0; fi < cnt; ++fi) my_dbs += s_dl[fi][tid];
        __syncthreads();                               // the stage and s_dl are free again
    }
    if (tid < n_sets * G && n_slabs > 0) {
#pragma unroll
        for (int e = 0; e < 4; ++e)
#pragma unroll
            for (int k = 0; k < MAX_CLASSES; ++k)
                if (k < C && 4 * cg + e < H) atomicAdd(&c.dW_s[k * H + 4 * cg + e], acc[e][k]);
    }
    if (tid < C && n_slabs > 0) atomicAdd(&c.db_s[tid], my_dbs);
    // lanes 0..3 of every warp hold row losses: fixed-order sum inside the warp, then over the warps
    my_loss += __shfl_down_sync(0xffffffffu, my_loss, 2);
    my_loss += __shfl_down_sync(0xffffffffu, my_loss, 1);
    if (lane == 0) warp_loss[wib] = my_loss;
    __syncthreads();
    if (tid == 0) {
        float t = 0.f;
        for (int w = 0; w < 8; ++w) t += warp_loss[w];
        c.loss_partial[blockIdx.x] = t;
    }
}

// ---- the same pass for the bf16 workloads (rows = the bf16 h of arena_bf), with the two small contractions on the tensor cores
// (warp-level mma.sync m16n8k16: the shapes are [64 rows x Hp] x [Hp x 8 classes] and [Hp x 64 rows] x [64 x 8],
// far too small for a tcgen05 tile).  States are bf16 already; W_s and dlog enter as a bf16 pair hi + lo
// (two MMAs), so the products carry about 16 mantissa bits and the sums are fp32.
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// x = hi + lo with hi, lo in bf16; packs (x0, x1) -> hi pair, lo pair
__device__ __forceinline__ void split_bf16x2(float x0, float x1, uint32_t& hi, uint32_t& lo) {
    const __nv_bfloat16 h0 = __float2bfloat16_rn(x0), h1 = __float2bfloat16_rn(x1);
    const __nv_bfloat162 hp = __halves2bfloat162(h0, h1);
    const __nv_bfloat162 lp = __floats2bfloat162_rn(x0 - __bfloat162float(h0), x1 - __bfloat162float(h1));
    hi = *reinterpret_cast<const uint32_t*>(&hp);
    lo = *reinterpret_cast<const uint32_t*>(&lp);
}

static const int LM_ROWS = 64;                         // rows per slab
static const int LM_KSTEPS_MAX = TC_HP_MAX / 16;       // k steps of the logits contraction
static const int LM_MT_MAX = (TC_HP_MAX / 16 + 7) / 8; // 16-unit tiles of dW_s per warp

__global__ void __launch_bounds__(256) rdf_loss_heads_mma_kernel(const DevCtx c) {
    if (c.ctl->status != 0) return;                    // an earlier kernel of this call failed: its lists and rows are not to be trusted
    extern __shared__ __align__(128) unsigned char slab_smem[];        // 2 stages of LM_ROWS rows, stride Hp * 2 + 16 bytes
    __shared__ __align__(8) uint64_t mbars[2];
    __shared__ __align__(16) float s_z[2][LM_ROWS][8];                 // partial logits of the two k halves
    __shared__ __align__(16) float s_dl[LM_ROWS][8];
    __shared__ int s_lab[2][LM_ROWS];
    __shared__ float warp_loss[8];
    const uint32_t F = c.ctl->frame_count.v, B = (uint32_t)c.B;
    const uint32_t n = F > B ? F - B : 0u, per = (n + gridDim.x - 1) / gridDim.x;
    const uint32_t f0 = min(F, B + blockIdx.x * per), f1 = min(F, f0 + per);
    const int n_slabs = (int)((f1 - f0 + LM_ROWS - 1) / LM_ROWS);
    const int tid = threadIdx.x, lane = tid % 32, warp = tid / 32, g = lane >> 2, t = lane & 3;
    const int H = c.H, Hp = c.Hp, C = c.n_classes;
    const bool dbs_from_pad = H < Hp;
    const uint32_t rowbytes = (uint32_t)Hp * 2u, stride = rowbytes + 16u, stage_bytes = LM_ROWS * stride;
    const uint32_t mbar = smem_u32(mbars), stage0 = smem_u32(slab_smem);
    int lab_next = 0;                                  // this thread's label of the slab that was issued last
    // stale rows of a short last slab must at least be finite: they meet dlog = 0 in the dW_s contraction
    for (uint32_t q = tid; q < 2 * stage_bytes / 16; q += 256) reinterpret_cast<uint4*>(slab_smem)[q] = make_uint4(0u, 0u, 0u, 0u);
    if (tid == 0) {
        mbar_init(mbar, 1);
        mbar_init(mbar + 8, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");       // the zeroes before the bulk copies that follow
    __syncthreads();
    auto issue = [&](int i) {
        const uint32_t fs = f0 + (uint32_t)i * LM_ROWS, cnt = min((uint32_t)LM_ROWS, f1 - fs), mb = mbar + 8 * (i & 1);
        if (tid == 0) asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(mb), "r"(cnt * rowbytes) : "memory");
        __syncthreads();                                               // the expectation is registered before any copy completes
        if (tid < (int)cnt) {
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(stage0 + (i & 1) * stage_bytes + tid * stride), "l"(c.arena_bf + (size_t)(fs + tid) * Hp), "r"(rowbytes), "r"(mb) : "memory");
            lab_next = __ldg(&c.label[(int)c.frames[fs + tid].arg]);       // two dependent loads: used one slab later
        }
    };
    // W_s fragments of this warp's k half: b0 = (k = 16 ks + 2t, +1; class g), b1 = (k + 8, + 9; class g), hi and lo
    const int ksteps = Hp / 16, khalf = (ksteps + 1) / 2, ks0 = (warp >> 2) * khalf, ks1 = min(ksteps, ks0 + khalf);
    uint32_t wb[(LM_KSTEPS_MAX + 1) / 2][4];
#pragma unroll
    for (int q = 0; q < (LM_KSTEPS_MAX + 1) / 2; ++q) {
        const int k = (ks0 + q) * 16 + 2 * t;
        float w[4] = {0.f, 0.f, 0.f, 0.f};
        if (ks0 + q < ks1 && g < C) {
            if (k < H) { w[0] = c.W_s[g * H + k]; w[1] = c.W_s[g * H + k + 1]; }         // H is a multiple of 4: k + 1 < H
            if (k + 8 < H) { w[2] = c.W_s[g * H + k + 8]; w[3] = c.W_s[g * H + k + 9]; }
        }
        split_bf16x2(w[0], w[1], wb[q][0], wb[q][2]);
        split_bf16x2(w[2], w[3], wb[q][1], wb[q][3]);
    }
    // dW_s accumulators: 16-unit tiles warp, warp + 8, warp + 16 of the Hp units; (unit g / g + 8, class 2t / 2t + 1)
    const int mtiles = Hp / 16;
    float acc[LM_MT_MAX][4];
#pragma unroll
    for (int m = 0; m < LM_MT_MAX; ++m)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[m][e] = 0.f;
    float my_loss = 0.f, my_dbs = 0.f;
    bool ok = true;
    if (n_slabs > 0) {
        issue(0);
        if (tid < LM_ROWS) s_lab[0][tid] = lab_next;
    }
    for (int i = 0; i < n_slabs; ++i) {
        if (i + 1 < n_slabs) issue(i + 1);             // its stage was released by the barrier that ended slab i - 1
        const uint32_t fs = f0 + (uint32_t)i * LM_ROWS, cnt = min((uint32_t)LM_ROWS, f1 - fs);
        ok = __syncthreads_and(mbar_wait(c, mbar + 8 * (i & 1), (uint32_t)(i >> 1) & 1u)) != 0;
        if (!ok) break;                                // the whole block agrees
        const uint32_t st = stage0 + (i & 1) * stage_bytes;
        // ---- logits: warp = (16-row tile warp & 3, k half warp >> 2)
        {
            float z[4] = {0.f, 0.f, 0.f, 0.f};
            const int mi = lane >> 3, ri = lane & 7;
            const uint32_t a_row = st + (uint32_t)((warp & 3) * 16 + (mi & 1) * 8 + ri) * stride + (uint32_t)(mi >> 1) * 16u;
#pragma unroll
            for (int q = 0; q < (LM_KSTEPS_MAX + 1) / 2; ++q) {
                if (ks0 + q >= ks1) break;
                uint32_t a[4];
                ldmatrix_x4(a, a_row + (uint32_t)(ks0 + q) * 32u);
                mma_bf16_16816(z, a, wb[q][0], wb[q][1]);
                mma_bf16_16816(z, a, wb[q][2], wb[q][3]);
            }
            float* zp = &s_z[warp >> 2][(warp & 3) * 16 + g][2 * t];
            zp[0] = z[0]; zp[1] = z[1];
            zp[8 * 8] = z[2]; zp[8 * 8 + 1] = z[3];    // row + 8
        }
        __syncthreads();
        // ---- softmax, loss, dlog: one thread per row
        if (tid < LM_ROWS) {
            float d[MAX_CLASSES];
#pragma unroll
            for (int k = 0; k < MAX_CLASSES; ++k) d[k] = 0.f;
            if (tid < (int)cnt) {
                const int lab = s_lab[i & 1][tid];
                float zr[MAX_CLASSES], m = -INFINITY;
#pragma unroll
                for (int k = 0; k < MAX_CLASSES; ++k)
                    if (k < C) {
                        zr[k] = s_z[0][tid][k] + s_z[1][tid][k] + __ldg(&c.b_s[k]);
                        m = fmaxf(m, zr[k]);
                    }
                float sum = 0.f, zl = 0.f;
#pragma unroll
                for (int k = 0; k < MAX_CLASSES; ++k)
                    if (k < C) {
                        sum += expf(zr[k] - m);
                        if (k == lab) zl = zr[k];
                    }
                my_loss += logf(sum) + m - zl;
#pragma unroll
                for (int k = 0; k < MAX_CLASSES; ++k) d[k] = k < C ? expf(zr[k] - m) / sum - (k == lab ? 1.f : 0.f) : 0.f;
                *reinterpret_cast<float4*>(c.dlog + (size_t)(fs + tid) * 8) = make_float4(d[0], d[1], d[2], d[3]);
                *reinterpret_cast<float4*>(c.dlog + (size_t)(fs + tid) * 8 + 4) = make_float4(d[4], d[5], d[6], d[7]);
            }
            *reinterpret_cast<float4*>(&s_dl[tid][0]) = make_float4(d[0], d[1], d[2], d[3]);      // rows past the end: zero
            *reinterpret_cast<float4*>(&s_dl[tid][4]) = make_float4(d[4], d[5], d[6], d[7]);
        }
        __syncthreads();
        // ---- dW_s^T [units x classes] += h^T [units x rows] dlog [rows x classes]
        {
            const int mi = lane >> 3, ri = lane & 7;
#pragma unroll
            for (int kk = 0; kk < LM_ROWS / 16; ++kk) {
                uint32_t bh0, bl0, bh1, bl1;
                split_bf16x2(s_dl[kk * 16 + 2 * t][g], s_dl[kk * 16 + 2 * t + 1][g], bh0, bl0);
                split_bf16x2(s_dl[kk * 16 + 2 * t + 8][g], s_dl[kk * 16 + 2 * t + 9][g], bh1, bl1);
                const uint32_t a_row = st + (uint32_t)(kk * 16 + (mi >> 1) * 8 + ri) * stride + (uint32_t)(mi & 1) * 16u;
#pragma unroll
                for (int m = 0; m < LM_MT_MAX; ++m) {
                    const int mt = warp + 8 * m;
                    if (mt >= mtiles) break;
                    uint32_t a[4];
                    ldmatrix_x4_trans(a, a_row + (uint32_t)mt * 32u);
                    mma_bf16_16816(acc[m], a, bh0, bh1);
                    mma_bf16_16816(acc[m], a, bl0, bl1);
                }
            }
        }
        // db_s = sum of dlog over the rows: with a pad column (H < Hp) the state rows carry the constant 1 in column H, so
        // row H of the contraction above is that sum; otherwise it is added up here
        if (!dbs_from_pad && tid < C)
            for (uint32_t fi = 0; fi < cnt; ++fi) my_dbs += s_dl[fi][tid];
        if (tid < LM_ROWS) s_lab[(i + 1) & 1][tid] = lab_next;      // labels of slab i + 1 (loaded while this slab was worked on)
        __syncthreads();                               // the stage, s_z and s_dl are free again
    }
    if (n_slabs > 0) {
#pragma unroll
        for (int m = 0; m < LM_MT_MAX; ++m) {
            const int mt = warp + 8 * m;
            if (mt >= mtiles) break;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int unit = mt * 16 + g + (e >> 1) * 8, cls = 2 * t + (e & 1);
                if (unit < H && cls < C) atomicAdd(&c.dW_s[cls * H + unit], acc[m][e]);
                else if (dbs_from_pad && unit == H && cls < C) atomicAdd(&c.db_s[cls], acc[m][e]);
            }
        }
        if (!dbs_from_pad && tid < C) atomicAdd(&c.db_s[tid], my_dbs);
    }
    // threads 0 .. 63 hold row losses: fixed-order sums inside the two warps, then over the warps
    for (int o = 16; o > 0; o >>= 1) my_loss += __shfl_down_sync(0xffffffffu, my_loss, o);
    if (lane == 0) warp_loss[warp] = my_loss;
    __syncthreads();
    if (tid == 0) c.loss_partial[blockIdx.x] = warp_loss[0] + warp_loss[1];
}

// Sum of the per-block partial losses in a fixed order (the same partials always give the same sum).
__global__ void __launch_bounds__(256) rdf_loss_final_kernel(const DevCtx c, int n_partials) {
    __shared__ double part[256];
    double t = 0.0;
    for (int i = threadIdx.x; i < n_partials; i += 256) t += (double)c.loss_partial[i];
    part[threadIdx.x] = t;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if ((int)threadIdx.x < o) part[threadIdx.x] += part[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        c.ctl->loss = (float)part[0];
        if (c.loss_out) *c.loss_out = (float)part[0];
        c.ctl->forward_status = c.ctl->status;      // what the gradient kernel checks before it starts
    }
}

// ---- reproducible mode: the loss head with sums that do not depend on how the invocations are spread over the blocks
// One warp per invocation.  Its logits are dot products in a fixed lane order (the value of an invocation is the same
// whichever warp computes it); the loss, dW_s and db_s are sums over all invocations and are accumulated as 64-bit
// fixed-point integers, per thread and then with integer atomics: exact, hence independent of the order.
// States: the bf16 h rows of arena_bf (tensor-core path).
__global__ void __launch_bounds__(256) rdf_loss_heads_exact_kernel(const DevCtx c) {
    if (c.ctl->status != 0) return;
    const uint32_t F = min(c.ctl->frame_count.v, c.frame_cap), B = (uint32_t)c.B;
    const int lane = threadIdx.x % 32, H = c.H, Hp = c.Hp, C = c.n_classes;
    const uint32_t warp = (blockIdx.x * blockDim.x + threadIdx.x) / 32, n_warps = gridDim.x * blockDim.x / 32;
    constexpr int MAXJ = TC_HP_MAX / 32;                               // hidden units per lane: j = lane + 32 q
    long long acc[MAX_CLASSES][MAXJ];
#pragma unroll
    for (int k = 0; k < MAX_CLASSES; ++k)
#pragma unroll
        for (int q = 0; q < MAXJ; ++q) acc[k][q] = 0;
    long long loss_acc = 0, dbs_acc = 0;                               // lane 0: the loss; lane k < C: db_s[k]
    for (uint32_t f = B + warp; f < F; f += n_warps) {
        float x[MAXJ], z[MAX_CLASSES];
#pragma unroll
        for (int q = 0; q < MAXJ; ++q) {
            const int j = lane + 32 * q;
            x[q] = j < H ? __bfloat162float(c.arena_bf[(size_t)f * Hp + j]) : 0.f;
        }
#pragma unroll
        for (int k = 0; k < MAX_CLASSES; ++k) {
            float t = 0.f;
            if (k < C) {
#pragma unroll
                for (int q = 0; q < MAXJ; ++q) {
                    const int j = lane + 32 * q;
                    if (j < H) t = fmaf(__ldg(&c.W_s[k * H + j]), x[q], t);
                }
                for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
                t += __ldg(&c.b_s[k]);
            }
            z[k] = t;
        }
        const int lab = __ldg(&c.label[(int)c.frames[f].arg]);
        float m = -INFINITY;
#pragma unroll
        for (int k = 0; k < MAX_CLASSES; ++k)
            if (k < C) m = fmaxf(m, z[k]);
        float sum = 0.f, zl = 0.f;
#pragma unroll
        for (int k = 0; k < MAX_CLASSES; ++k)
            if (k < C) {
                sum += expf(z[k] - m);
                if (k == lab) zl = z[k];
            }
        float d[MAX_CLASSES];
#pragma unroll
        for (int k = 0; k < MAX_CLASSES; ++k) d[k] = k < C ? expf(z[k] - m) / sum - (k == lab ? 1.f : 0.f) : 0.f;
        if (lane == 0) {
            loss_acc += to_fix(logf(sum) + m - zl);
            *reinterpret_cast<float4*>(c.dlog + (size_t)f * 8) = make_float4(d[0], d[1], d[2], d[3]);
            *reinterpret_cast<float4*>(c.dlog + (size_t)f * 8 + 4) = make_float4(d[4], d[5], d[6], d[7]);
        }
#pragma unroll
        for (int k = 0; k < MAX_CLASSES; ++k) {
            if (k >= C) continue;
            if (lane == k) dbs_acc += to_fix(d[k]);
#pragma unroll
            for (int q = 0; q < MAXJ; ++q) acc[k][q] += to_fix(d[k] * x[q]);
        }
    }
#pragma unroll
    for (int k = 0; k < MAX_CLASSES; ++k) {
        if (k >= C) continue;
#pragma unroll
        for (int q = 0; q < MAXJ; ++q) {
            const int j = lane + 32 * q;
            if (j < H && acc[k][q] != 0) fix_add(&c.head_fix[k * H + j], acc[k][q]);
        }
    }
    if (lane < C && dbs_acc != 0) fix_add(&c.head_fix[C * H + lane], dbs_acc);
    if (lane == 0 && loss_acc != 0) fix_add(&c.head_fix[C * (H + 1)], loss_acc);
}

// the fixed-point sums as fp32: dW_s, db_s, the loss
__global__ void __launch_bounds__(256) rdf_head_convert_kernel(const DevCtx c) {
    const int C = c.n_classes, H = c.H, n = C * (H + 1) + 1;
    const int q = blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= n) return;
    if (q == n - 1) {
        // (this thread also closes the forward pass: what the gradient kernel checks before it starts)
        const float loss = from_fix(c.head_fix[q]);
        c.ctl->loss = loss;
        if (c.loss_out) *c.loss_out = loss;
        c.ctl->forward_status = c.ctl->status;
        return;
    }
    if (c.ctl->status != 0) return;
    const float v = from_fix(c.head_fix[q]);
    if (q < C * H) c.dW_s[q] = v;
    else c.db_s[q - C * H] = v;
}

// the embedding gradient from its fixed-point sums
__global__ void __launch_bounds__(256) rdf_de_convert_kernel(const DevCtx c) {
    if (c.ctl->status != 0) return;
    const size_t total = (size_t)c.V * c.D / 2;                        // two elements per thread step (D is a multiple of 4)
    for (size_t q = (size_t)blockIdx.x * blockDim.x + threadIdx.x; q < total; q += (size_t)gridDim.x * blockDim.x) {
        const longlong2 v = *reinterpret_cast<const longlong2*>(c.dE_fix + 2 * q);
        *reinterpret_cast<float2*>(c.dE + 2 * q) = make_float2(from_fix(v.x), from_fix(v.y));
    }
}

// ----------------------------------------------------------- backward waves
// What a thread needs to know about an invocation before it touches its rows; all of it is left
// behind by the forward pass and the loss head, so it can be fetched one step ahead.
struct FrameMeta {
    uint32_t l, r, parent;
    float4 d0, d1;
};
__device__ __forceinline__ FrameMeta load_meta(const DevCtx& c, uint32_t t) {
    FrameMeta m;
    m.l = c.op_l[t]; m.r = c.op_r[t]; m.parent = c.frames[t].parent;
    m.d0 = *reinterpret_cast<const float4*>(c.dlog + (size_t)t * 8);
    m.d1 = *reinterpret_cast<const float4*>(c.dlog + (size_t)t * 8 + 4);
    return m;
}

// A (bf16 TreeRNN), the invocations called from `result` (no gradient comes in from a caller), one per
// 8 lanes and step: dh = W_s^T dlog; cell: dz = dh * (1 - h^2) as the bf16 operand row of the
// contractions; leaf: dE[tok] += dh.  A lane owns 8 consecutive hidden units per 64.  Every other
// invocation gets the same treatment from the epilogue of its caller's operand-gradient tile.
__device__ __forceinline__ void backward_frames_tc(const DevCtx& c, uint32_t t0, uint32_t end, uint32_t stride, int sl) {
    const int H = c.H, Hp = c.Hp, C = c.n_classes;
    constexpr int NQ = TC_HP_MAX / 64;
    if (t0 >= end) return;
    FrameMeta m = load_meta(c, t0);
    for (uint32_t t = t0; t < end; t += stride) {
        const bool leaf = m.l == LEAF_MARK;
        const uint32_t tok = m.r;
        const uint32_t pos = leaf ? 0u : c.cell_pos[t];               // the cell's dz row
        const float dl[MAX_CLASSES] = {m.d0.x, m.d0.y, m.d0.z, m.d0.w, m.d1.x, m.d1.y, m.d1.z, m.d1.w};
        uint4 hv[NQ];
#pragma unroll
        for (int q = 0; q < NQ; ++q) {
            const int j = sl * 8 + 64 * q;
            hv[q] = make_uint4(0u, 0u, 0u, 0u);
            if (!leaf && j < Hp) hv[q] = *reinterpret_cast<const uint4*>(c.arena_bf + (size_t)t * Hp + j);
        }
        if (t + stride < end) m = load_meta(c, t + stride);
#pragma unroll
        for (int q = 0; q < NQ; ++q) {
            const int j = sl * 8 + 64 * q;
            if (j >= Hp) continue;
            float dh[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int k = 0; k < MAX_CLASSES; ++k)
                if (k < C) {
                    if (j < H) {
                        const float4 w = __ldg(reinterpret_cast<const float4*>(&c.W_s[k * H + j]));
                        dh[0] = fmaf(w.x, dl[k], dh[0]); dh[1] = fmaf(w.y, dl[k], dh[1]);
                        dh[2] = fmaf(w.z, dl[k], dh[2]); dh[3] = fmaf(w.w, dl[k], dh[3]);
                    }
                    if (j + 4 < H) {
                        const float4 w = __ldg(reinterpret_cast<const float4*>(&c.W_s[k * H + j + 4]));
                        dh[4] = fmaf(w.x, dl[k], dh[4]); dh[5] = fmaf(w.y, dl[k], dh[5]);
                        dh[6] = fmaf(w.z, dl[k], dh[6]); dh[7] = fmaf(w.w, dl[k], dh[7]);
                    }
                }
            if (leaf && c.dE_fix) {                              // reproducible mode: exact integer sums
                long long* de = c.dE_fix + (size_t)tok * c.D + j;
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    if (j + i < H) fix_add(de + i, to_fix(dh[i]));
            } else if (leaf) {
                float* de = c.dE + (size_t)tok * c.D + j;
                if (j < H) atomicAdd(reinterpret_cast<float4*>(de), make_float4(dh[0], dh[1], dh[2], dh[3]));
                if (j + 4 < H) atomicAdd(reinterpret_cast<float4*>(de + 4), make_float4(dh[4], dh[5], dh[6], dh[7]));
            } else {
                float x[8];
                unpack_bf8(hv[q], x);
#pragma unroll
                for (int i = 0; i < 8; ++i) dh[i] *= 1.f - x[i] * x[i];      // pad columns: dh = 0 and h = 0, so dz = 0
                __align__(16) __nv_bfloat162 pk[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) pk[i] = __floats2bfloat162_rn(dh[2 * i], dh[2 * i + 1]);
                *reinterpret_cast<uint4*>(c.dz_bf + (size_t)pos * Hp + j) = *reinterpret_cast<const uint4*>(pk);
            }
        }
    }
}

// A (fp32 TreeRNN), one invocation per 8 lanes and step; dz (cell) replaces the incoming gradient.
__device__ __forceinline__ void backward_frames_f32(const DevCtx& c, uint32_t t0, uint32_t end, uint32_t stride, int sl) {
    const int H = c.H, C = c.n_classes;
    if (t0 >= end) return;
    FrameMeta m = load_meta(c, t0);
    for (uint32_t t = t0; t < end; t += stride) {
        const bool from_result = m.parent < (uint32_t)c.B, leaf = m.l == LEAF_MARK;
        const uint32_t tok = m.r;
        const float dl[MAX_CLASSES] = {m.d0.x, m.d0.y, m.d0.z, m.d0.w, m.d1.x, m.d1.y, m.d1.z, m.d1.w};
        if (t + stride < end) m = load_meta(c, t + stride);
        float* g = c.dhp + (size_t)t * H;
        const float* h = c.arena + (size_t)t * H;
#pragma unroll 4
        for (int j = sl * 4; j < H; j += 32) {
            float4 dh = ldcg4(g + j);                    // (not used for an invocation called from `result`)
            const float4 hv = leaf ? make_float4(0.f, 0.f, 0.f, 0.f) : *reinterpret_cast<const float4*>(h + j);
            if (from_result) dh = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int k = 0; k < MAX_CLASSES; ++k)
                if (k < C) {
                    const float4 w = __ldg(reinterpret_cast<const float4*>(&c.W_s[k * H + j]));
                    dh.x = fmaf(w.x, dl[k], dh.x); dh.y = fmaf(w.y, dl[k], dh.y);
                    dh.z = fmaf(w.z, dl[k], dh.z); dh.w = fmaf(w.w, dl[k], dh.w);
                }
            if (leaf) {
                atomicAdd(reinterpret_cast<float4*>(c.dE + (size_t)tok * c.D + j), dh);
            } else {
                dh.x *= 1.f - hv.x * hv.x; dh.y *= 1.f - hv.y * hv.y;
                dh.z *= 1.f - hv.z * hv.z; dh.w *= 1.f - hv.w * hv.w;
                *reinterpret_cast<float4*>(g + j) = dh;
            }
        }
    }
}

// A (TreeLSTM): the gate gradients replace the retained gates; dc goes straight to the callee frames.
// One invocation t per warp.
__device__ __forceinline__ void lstm_backward_frame(const DevCtx& c, uint32_t t, int lane) {
    const int H = c.H, C = c.n_classes, S = c.S;
    {
        const uint32_t parent = __ldcg(&c.frames[t].parent);
        const bool from_result = parent < (uint32_t)c.B;
        const uint32_t l = __ldcg(&c.op_l[t]), r = __ldcg(&c.op_r[t]);
        const bool leaf = l == LEAF_MARK;
        float dl[MAX_CLASSES];
#pragma unroll
        for (int k = 0; k < MAX_CLASSES; ++k) dl[k] = __ldcg(&c.dlog[(size_t)t * 8 + k]);
        const float* g = c.dhp + (size_t)t * S;
        const float* st = c.arena + (size_t)t * S;
        float* gt = c.gates + (size_t)t * c.G;
        // 128-bit accesses: four hidden units per lane and step
        auto ld = [](const float* p) { const float4 v = ldcg4(p); return v; };
        auto st4 = [](float* p, const float (&v)[4]) { *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]); };
        const bool keep_f32 = c.dg_bf == nullptr;       // bf16 path: the gate gradients live on as bf16 operand rows only
        auto stb = [&](int gate, int j, const float (&v)[4]) {
            if (!c.dg_bf) return;
            __nv_bfloat162 lo = __floats2bfloat162_rn(v[0], v[1]), hi = __floats2bfloat162_rn(v[2], v[3]);
            uint2 pk;
            pk.x = *reinterpret_cast<uint32_t*>(&lo);
            pk.y = *reinterpret_cast<uint32_t*>(&hi);
            *reinterpret_cast<uint2*>(c.dg_bf + (size_t)t * 5 * c.Hp + gate * c.Hp + j) = pk;
        };
        for (int j = lane * 4; j < H; j += 128) {
            const float4 z4 = make_float4(0.f, 0.f, 0.f, 0.f);
            const float4 dh4 = from_result ? z4 : ld(g + j), dc4 = from_result ? z4 : ld(g + H + j), c4 = ld(st + H + j);
            float dh[4] = {dh4.x, dh4.y, dh4.z, dh4.w};
            const float dci[4] = {dc4.x, dc4.y, dc4.z, dc4.w}, cc[4] = {c4.x, c4.y, c4.z, c4.w};
#pragma unroll
            for (int k = 0; k < MAX_CLASSES; ++k)
                if (k < C) {
                    const float4 w = __ldg(reinterpret_cast<const float4*>(&c.W_s[k * H + j]));
                    dh[0] = fmaf(w.x, dl[k], dh[0]); dh[1] = fmaf(w.y, dl[k], dh[1]);
                    dh[2] = fmaf(w.z, dl[k], dh[2]); dh[3] = fmaf(w.w, dl[k], dh[3]);
                }
            if (leaf) {
                const float4 a4 = ld(gt + j), o4 = ld(gt + H + j), u4 = ld(gt + 2 * H + j);
                const float gi[4] = {a4.x, a4.y, a4.z, a4.w}, go[4] = {o4.x, o4.y, o4.z, o4.w}, gu[4] = {u4.x, u4.y, u4.z, u4.w};
                float g0[4], g1[4], g2[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float tc = tanhf(cc[e]);
                    const float dc = dci[e] + dh[e] * go[e] * (1.f - tc * tc);
                    g0[e] = dc * gu[e] * gi[e] * (1.f - gi[e]);
                    g1[e] = dh[e] * tc * go[e] * (1.f - go[e]);
                    g2[e] = dc * gi[e] * (1.f - gu[e] * gu[e]);
                }
                if (keep_f32) { st4(gt + j, g0); st4(gt + H + j, g1); st4(gt + 2 * H + j, g2); }
                stb(0, j, g0); stb(1, j, g1); stb(2, j, g2);
            } else {
                const float4 a4 = ld(gt + j), l4 = ld(gt + H + j), r4 = ld(gt + 2 * H + j), o4 = ld(gt + 3 * H + j), u4 = ld(gt + 4 * H + j);
                const float4 cl4 = ld(c.arena + (size_t)l * S + H + j), cr4 = ld(c.arena + (size_t)r * S + H + j);
                const float gi[4] = {a4.x, a4.y, a4.z, a4.w}, fl[4] = {l4.x, l4.y, l4.z, l4.w}, fr[4] = {r4.x, r4.y, r4.z, r4.w};
                const float go[4] = {o4.x, o4.y, o4.z, o4.w}, gu[4] = {u4.x, u4.y, u4.z, u4.w};
                const float cl[4] = {cl4.x, cl4.y, cl4.z, cl4.w}, cr[4] = {cr4.x, cr4.y, cr4.z, cr4.w};
                float g0[4], g1[4], g2[4], g3[4], g4[4], dl_[4], dr_[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float tc = tanhf(cc[e]);
                    const float dc = dci[e] + dh[e] * go[e] * (1.f - tc * tc);
                    g0[e] = dc * gu[e] * gi[e] * (1.f - gi[e]);
                    g1[e] = dc * cl[e] * fl[e] * (1.f - fl[e]);
                    g2[e] = dc * cr[e] * fr[e] * (1.f - fr[e]);
                    g3[e] = dh[e] * tc * go[e] * (1.f - go[e]);
                    g4[e] = dc * gi[e] * (1.f - gu[e] * gu[e]);
                    dl_[e] = dc * fl[e];
                    dr_[e] = dc * fr[e];
                }
                if (keep_f32) { st4(gt + j, g0); st4(gt + H + j, g1); st4(gt + 2 * H + j, g2); st4(gt + 3 * H + j, g3); st4(gt + 4 * H + j, g4); }
                stb(0, j, g0); stb(1, j, g1); stb(2, j, g2); stb(3, j, g3); stb(4, j, g4);
                st4(c.dhp + (size_t)l * S + H + j, dl_);
                st4(c.dhp + (size_t)r * S + H + j, dr_);
            }
        }
        if (c.dg_bf)                      // pad columns of every gate block are zero
            for (int q = lane; q < (leaf ? 3 : 5) * (c.Hp - H); q += 32)
                c.dg_bf[(size_t)t * 5 * c.Hp + (q / (c.Hp - H)) * c.Hp + H + q % (c.Hp - H)] = __float2bfloat16_rn(0.f);
    }
}

// B: [dh_l ; dh_r] = W^T dg for the cells all_cells[first, first + n).  dg of cell t is the row
//    A[t * lda .. + Kdim): dz (TreeRNN, Kdim = H) or the five gate gradients (TreeLSTM, Kdim = 5H).
__device__ void backward_operand_tiles(const DevCtx& c, GemmSmem& sm, uint32_t first, uint32_t n_items,
                                       const float* A, int lda, int Kdim) {
    const int H = c.H, K2 = 2 * c.H, S = c.S;
    const int tiles_m = (n_items + TM - 1) / TM, tiles_n = (K2 + TN - 1) / TN;
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
    const int arow_l = threadIdx.x / 4, ak = (threadIdx.x % 4) * 4;     // A loader: row, 4 consecutive k
    const int bk = threadIdx.x / 16, bn = (threadIdx.x % 16) * 4;       // B loader: k, 4 consecutive columns
    for (int tile = blockIdx.x; tile < tiles_m * tiles_n; tile += gridDim.x) {
        const int tm = tile / tiles_n, tn = tile % tiles_n;
        const int row0 = tm * TM, col0 = tn * TN;
        const int arow = row0 + arow_l;
        const float* dz = nullptr;
        if (arow < (int)n_items) dz = A + (size_t)__ldcg(&c.all_cells[first + arow]) * lda;
        float acc[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
        // the operands of step k0 + TK are on their way (registers) while step k0 is multiplied
        auto fetch = [&](int k0, float4& a, float4& b) {
            a = make_float4(0.f, 0.f, 0.f, 0.f); b = a;
            if (dz && k0 + ak < Kdim) a = ldcg4(dz + k0 + ak);
            if (k0 + bk < Kdim && col0 + bn < K2)
                b = __ldg(reinterpret_cast<const float4*>(c.W + (size_t)(k0 + bk) * K2 + col0 + bn));
        };
        float4 a, b;
        fetch(0, a, b);
        for (int k0 = 0; k0 < Kdim; k0 += TK) {
            __syncthreads();
            sm.As[ak + 0][arow_l] = a.x; sm.As[ak + 1][arow_l] = a.y; sm.As[ak + 2][arow_l] = a.z; sm.As[ak + 3][arow_l] = a.w;
            *reinterpret_cast<float4*>(&sm.Bs[bk][bn]) = b;
            __syncthreads();
            if (k0 + TK < Kdim) fetch(k0 + TK, a, b);
            gemm_tile_step(sm, tx, ty, acc);
        }
        const int col = col0 + tx * 4;
        if (col < K2) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int row = row0 + ty * 4 + i;
                if (row < (int)n_items) {
                    const uint32_t t = __ldcg(&c.all_cells[first + row]);
                    const uint32_t child = col < H ? __ldcg(&c.op_l[t]) : __ldcg(&c.op_r[t]);
                    const int cc = col < H ? col : col - H;
                    *reinterpret_cast<float4*>(c.dhp + (size_t)child * S + cc) =
                        make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
                }
            }
        }
    }
}

// Narrow waves: an 8 cell x 32 column patch of [dh_l ; dh_r] = W^T dz per block step;
// thread = (cell, 4 columns, quarter of the contraction over j).  The thread that ends up with the four
// sums finishes the callee they belong to right away (what the per-invocation pass would do one wave
// later): dh += W_s^T dlog; a cell callee gets dz = dh (1 - h^2) in place of its incoming gradient, a leaf
// callee adds dh to dE[tok].  What it needs of the callee is fetched before the contraction starts.
// wres: this block's resident 32 columns of W in shared memory (or nullptr) as float4 [j][4-column group],
// the columns of the column group blockIdx.x % units_n.
__device__ void backward_operand_thin(const DevCtx& c, float* zs, const float4* wres, uint32_t first, uint32_t n_items) {
    // zs: shared staging for the 8 dz rows of the patch (8 x H floats), 768 floats of partial sums, 8 records
    const int H = c.H, K2 = 2 * c.H, C = c.n_classes;
    float* red = zs + 8 * H;
    uint4* s_rec = reinterpret_cast<uint4*>(red + 768);                    // {cell, left callee, right callee, valid}
    const int units_n = (K2 + 31) / 32, units = ((n_items + 7) / 8) * units_n;
    const int o = threadIdx.x & 63, jq = threadIdx.x >> 6, rr = o >> 3, c4 = o & 7;
    const int jlen = (H + 3) / 4;
    for (int unit = blockIdx.x; unit < units; unit += gridDim.x) {
        const int row0 = (unit / units_n) * 8;
        if (threadIdx.x < 8) {
            uint4 rec = make_uint4(0u, 0u, 0u, 0u);
            if (row0 + (int)threadIdx.x < (int)n_items) {
                rec.x = __ldcg(&c.all_cells[first + row0 + threadIdx.x]);
                rec.y = c.op_l[rec.x]; rec.z = c.op_r[rec.x]; rec.w = 1u;
            }
            s_rec[threadIdx.x] = rec;
        }
        for (int p = threadIdx.x; p < 8 * (H / 4); p += blockDim.x) {
            const int r = p / (H / 4), k = (p % (H / 4)) * 4;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (row0 + r < (int)n_items) v = ldcg4(c.dhp + (size_t)__ldcg(&c.all_cells[first + row0 + r]) * H + k);
            *reinterpret_cast<float4*>(zs + r * H + k) = v;
        }
        __syncthreads();
        const int row = row0 + rr, col = (unit % units_n) * 32 + c4 * 4;
        const bool live = row < (int)n_items && col < K2;
        // the callee this thread will finish, fetched while the contraction runs
        const int cc = col < H ? col : col - H;
        uint32_t child = 0, child_l = LEAF_MARK, child_tok = 0;
        float4 d0 = make_float4(0.f, 0.f, 0.f, 0.f), d1 = d0, hv = d0;
        if (jq == 0 && live) {
            const uint4 rec = s_rec[rr];
            child = col < H ? rec.y : rec.z;
            child_l = c.op_l[child]; child_tok = c.op_r[child];
            d0 = *reinterpret_cast<const float4*>(c.dlog + (size_t)child * 8);
            d1 = *reinterpret_cast<const float4*>(c.dlog + (size_t)child * 8 + 4);
            hv = *reinterpret_cast<const float4*>(c.arena + (size_t)child * H + cc);
        }
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        if (live) {
            const float* dz = zs + rr * H;
            const int j0 = jq * jlen, j1 = min(H, j0 + jlen);
            if (wres && unit % units_n == (int)(blockIdx.x % units_n)) {
#pragma unroll 8
                for (int j = j0; j < j1; ++j) {
                    const float d = dz[j];
                    const float4 w = wres[j * 8 + c4];
                    acc.x = fmaf(d, w.x, acc.x); acc.y = fmaf(d, w.y, acc.y);
                    acc.z = fmaf(d, w.z, acc.z); acc.w = fmaf(d, w.w, acc.w);
                }
            } else {
#pragma unroll 8
                for (int j = j0; j < j1; ++j) {
                    const float d = dz[j];
                    const float4 w = __ldg(reinterpret_cast<const float4*>(c.W + (size_t)j * K2 + col));
                    acc.x = fmaf(d, w.x, acc.x); acc.y = fmaf(d, w.y, acc.y);
                    acc.z = fmaf(d, w.z, acc.z); acc.w = fmaf(d, w.w, acc.w);
                }
            }
        }
        if (jq > 0) *reinterpret_cast<float4*>(red + ((jq - 1) * 64 + o) * 4) = acc;
        __syncthreads();
        if (jq == 0 && live) {
#pragma unroll
            for (int q = 0; q < 3; ++q) {
                const float4 p = *reinterpret_cast<const float4*>(red + (q * 64 + o) * 4);
                acc.x += p.x; acc.y += p.y; acc.z += p.z; acc.w += p.w;
            }
            const float dl[MAX_CLASSES] = {d0.x, d0.y, d0.z, d0.w, d1.x, d1.y, d1.z, d1.w};
#pragma unroll
            for (int k = 0; k < MAX_CLASSES; ++k)
                if (k < C) {
                    const float4 w = __ldg(reinterpret_cast<const float4*>(&c.W_s[k * H + cc]));
                    acc.x = fmaf(w.x, dl[k], acc.x); acc.y = fmaf(w.y, dl[k], acc.y);
                    acc.z = fmaf(w.z, dl[k], acc.z); acc.w = fmaf(w.w, dl[k], acc.w);
                }
            if (child_l == LEAF_MARK) {
                atomicAdd(reinterpret_cast<float4*>(c.dE + (size_t)child_tok * c.D + cc), acc);
            } else {
                acc.x *= 1.f - hv.x * hv.x; acc.y *= 1.f - hv.y * hv.y;
                acc.z *= 1.f - hv.z * hv.z; acc.w *= 1.f - hv.w * hv.w;
                *reinterpret_cast<float4*>(c.dhp + (size_t)child * H + cc) = acc;
            }
        }
        __syncthreads();
    }
}

template <bool TC, bool RNN32 = false>         // RNN32: the fp32 TreeRNN alone, two blocks per SM (see rdf_operator_kernel)
__global__ void __launch_bounds__(TC ? TC_THREADS : 256, RNN32 ? 2 : 1) rdf_backward_kernel(const __grid_constant__ DevCtx c) {
    const bool lstm = RNN32 ? false : c.lstm != 0;
    __shared__ typename std::conditional<TC, TcShared, LstmSmem>::type smem;   // fp32: tiles use the first part; thin patches stage rows in it
    extern __shared__ unsigned char dyn_smem[];                      // tensor-core path: resident W^T slice + A stages
    if (c.ctl->forward_status != 0) return;                          // the forward pass failed: nothing to differentiate
    TcState tc;
    if constexpr (TC) {
        if (lstm) tc_setup(tc, smem, dyn_smem, (2 * c.Hp + TC_LSTM_BWD_NS - 1) / TC_LSTM_BWD_NS, c.WTp, 5 * c.Hp, TC_LSTM_BWD_NS, nullptr, 0, 0, 2 * c.Hp);
        else tc_setup(tc, smem, dyn_smem, 8, c.WTp, c.Hp, c.Hp / 4);
        tc_setup_epilogue(c, tc, smem, true);
    }
    // fp32 TreeRNN, narrow waves: this block's 32 columns of W stay in shared memory for all waves
    const float4* wres = nullptr;
    if constexpr (!TC) {
        if (!lstm && c.H <= THIN_RESIDENT_MAX_H) {
            float4* wr = reinterpret_cast<float4*>(dyn_smem);
            const int K2 = 2 * c.H, units_n = (K2 + 31) / 32, cg0 = blockIdx.x % units_n;
            for (int q = threadIdx.x; q < c.H * 8; q += blockDim.x) {
                const int j = q / 8, col = cg0 * 32 + (q % 8) * 4;
                wr[q] = col < K2 ? __ldg(reinterpret_cast<const float4*>(c.W + (size_t)j * K2 + col)) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
            __syncthreads();
            wres = wr;
        }
    }
    const int lane = threadIdx.x % 32, wib = threadIdx.x / 32, n_warps = blockDim.x / 32;
    uint32_t generation = 0, wave = 0;
    long long cyc_a = 0, cyc_c = 0, cyc_b = 0, t_mark = clock64();
    auto lap = [&](long long& acc) {
        const long long now = clock64();
        acc += now - t_mark;
        t_mark = now;
    };
    // Gradient wave k re-enters the invocations of call depth k (the k-th scheduler wave that made calls): frame ids
    // are handed out in wave order, so they are one id range [f0, f1) and their rows are consecutive in memory; the
    // cells among them are all_cells[first, end).
    const uint32_t nw = min(c.ctl->n_depth_waves, c.wave_cap);
    bool callees_done = false;        // the previous wave's contraction has already finished this wave's invocations
    uint4 wv = nw ? c.wave_marks[0] : make_uint4(0u, 0u, 0u, 0u);
    // clustered gradient pass (fp32 TreeRNN, deep recursions): this kernel runs the wide call depths only, up to d_split
    const bool clustered = !TC && !lstm && depth_groups(c) > 1u;
    const uint32_t d_split = clustered ? c.ctl->d_split : 0u;
    for (uint32_t k = 0; k < nw; ++k) {
        const uint4 cur = wv;
        if (k + 1 < nw) wv = c.wave_marks[k + 1];                    // in flight during this wave
        const uint32_t f0 = min(cur.x, c.frame_cap), f1 = min(cur.y, c.frame_cap);
        if (f1 <= f0) continue;
        if (clustered && (__ldcg(&c.frames[f0].label) >> FRAME_WAVE_SHIFT) + 1u > d_split) {
            // The first depth of the clusters: they expect the invocations of a depth finished (gradient of the loss head
            // added, dz in place of dh), as the contraction of the depth above leaves them; do that here where it has not.
            if (!callees_done) {
                const uint32_t n = f1 - f0;
                const uint32_t per = ((n + gridDim.x - 1) / gridDim.x + 31u) & ~31u;
                const unsigned long long c0l = (unsigned long long)f0 + (unsigned long long)blockIdx.x * per;
                const uint32_t c0 = (uint32_t)min(c0l, (unsigned long long)f1), c1 = (uint32_t)min(c0l + per, (unsigned long long)f1);
                backward_frames_f32(c, c0 + wib * 4 + lane / 8, c1, 4 * n_warps, lane % 8);
            }
            break;
        }
        ++wave;
        // ---- A: per-invocation work, a contiguous piece of the range per block.  (bf16 TreeRNN: only the
        //      invocations called from `result` -- further down the epilogue of B does this work for the callees;
        //      fp32 TreeRNN: not after a wave of narrow patches, which do the same.)
        if (!(TC && !lstm && k > 0) && !callees_done) {
            const uint32_t n = f1 - f0;
            const uint32_t per = ((n + gridDim.x - 1) / gridDim.x + 31u) & ~31u;
            const unsigned long long c0l = (unsigned long long)f0 + (unsigned long long)blockIdx.x * per;
            const uint32_t c0 = (uint32_t)min(c0l, (unsigned long long)f1), c1 = (uint32_t)min(c0l + per, (unsigned long long)f1);
            bool done_a = false;
            if constexpr (!RNN32) {
                if (lstm) {
                    for (uint32_t t = c0 + wib; t < c1; t += n_warps) lstm_backward_frame(c, t, lane);
                    done_a = true;
                }
            }
            if (done_a) {
            } else if constexpr (TC) {
                backward_frames_tc(c, c0 + wib * 4 + lane / 8, c1, 4 * n_warps, lane % 8);
                asm volatile("fence.proxy.async;" ::: "memory");       // its dz rows are read by tile copies after the barrier
            } else {
                backward_frames_f32(c, c0 + wib * 4 + lane / 8, c1, 4 * n_warps, lane % 8);
            }
            __syncthreads();
            lap(cyc_a);
            if (!grid_barrier(c, &c.ctl->bar2.v, generation)) break;
            lap(cyc_b);
        }
        // ---- B: operand gradients of the wave's cells, handed to the frames of the calls they made
        const uint32_t first = min(cur.z, c.frame_cap), end = min(cur.w, c.frame_cap);
        bool thin = false;
        if (end > first) {
            if constexpr (TC) {
                if (lstm) tc_pipe<TC_LSTM_BWD, TC_STAGES_LSTM_BWD>(c, tc, smem, first, end - first);
                else tc_pipe<TC_RNN_BWD, TC_STAGES_RNN_BWD>(c, tc, smem, first, end - first);
            } else {
                if (lstm) backward_operand_tiles(c, *reinterpret_cast<GemmSmem*>(&smem), first, end - first, c.gates, c.G, 5 * c.H);
                else if (c.H <= 512 && ((end - first + 7) / 8) * ((2 * c.H + 31) / 32) <= 2 * gridDim.x) {
                    backward_operand_thin(c, reinterpret_cast<float*>(&smem), wres, first, end - first);   // 8 x H + 800 floats <= 26 KB
                    thin = true;
                } else backward_operand_tiles(c, *reinterpret_cast<GemmSmem*>(&smem), first, end - first, c.dhp, c.H, c.H);
            }
            __syncthreads();
            lap(cyc_c);
            if (!grid_barrier(c, &c.ctl->bar2.v, generation)) break;
            lap(cyc_b);
        }
        callees_done = thin;
    }
    if constexpr (TC) tc_teardown(tc);
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        c.ctl->waves_backward = wave;
        c.ctl->cyc[3] = cyc_a; c.ctl->cyc[4] = cyc_c; c.ctl->cyc[5] = cyc_b;
    }
}

// ===========================================================================
// fp32 TreeRNN gradient waves without a grid barrier: one thread-block cluster per group of instances
// ===========================================================================
// The counterpart of rdf_operator_cluster_kernel for the reverse pass.  The cells are grouped by (cluster of their
// instance, call depth); a cluster runs the depths below the split one after the other for its own instances and
// meets at the hardware cluster barrier only.  Per cell: [dh_l ; dh_r] = W^T dz; the blocks of a cluster split the 2H
// output columns (their part of W stays in shared memory), a block step takes CS cells, thread = (column, slice of the
// contraction index); the thread that adds the slices up finishes the callee of its column (adds W_s^T dlog; a cell
// callee gets dz = dh (1 - h^2) as its row, a leaf callee adds dh to dE[tok]) -- what it needs of the callee is
// fetched before the contraction starts.  Rows travel between the blocks through L2, ordered by the barrier.
static const int BWD_CLUSTER_THREADS = 512;
template <int CPC, int CS>                     // columns per block; cells per step = slices of the contraction index (CPC x CS threads work)
__global__ void __launch_bounds__(BWD_CLUSTER_THREADS, 1) rdf_backward_cluster_kernel(const __grid_constant__ DevCtx c) {
    extern __shared__ __align__(16) unsigned char dyn_smem[];
    // every block takes the same decision from the same words (the kernels before this one are complete)
    if (c.ctl->forward_status != 0 || c.ctl->status != 0 || depth_groups(c) <= 1u) return;
    const int H = c.H, K2 = 2 * c.H, C = c.n_classes;
    const int rank = blockIdx.x % CLUSTER_CTAS, group = blockIdx.x / CLUSTER_CTAS;
    const int j0 = rank * CPC;                                         // first of this block's output columns (of 2H)
    float* wres = reinterpret_cast<float*>(dyn_smem);                  // [H][CPC]: W[j][j0 + jj]
    float* zs = wres + (size_t)H * CPC;                                // [2][CS][H]: dz rows, double buffered
    float* part = zs + (size_t)2 * CS * H;                             // [CS slices][CS cells][CPC]
    uint4* s_rec = reinterpret_cast<uint4*>(part + (size_t)CS * CS * CPC);   // [2][CS]: {cell, left callee, right callee, -}; then the ring
    for (int q = threadIdx.x; q < H * CPC; q += blockDim.x) {
        const int j = q / CPC, jj = q % CPC;
        wres[q] = j0 + jj < K2 ? __ldg(&c.W[(size_t)j * K2 + j0 + jj]) : 0.f;
    }
    __syncthreads();
    const uint32_t stride = bucket_stride(c, 1), top = stride - 1u;
    const uint32_t* ends = c.height_ends + (size_t)group * stride;     // ends[d]: end of (group, depth d); ends[0]: start of the group
    const int jj = threadIdx.x % CPC, ks = threadIdx.x / CPC;          // column; slice of the contraction (then: cell)
    const bool active = ks < CS;
    const int col = j0 + jj, cc = col < H ? col : col - H;
    const int klen = ((H + CS - 1) / CS + 3) & ~3, k_begin = ks * klen, k_end = min(H, k_begin + klen);
    const int pieces = CS * (H / 4);
    auto stage = [&](int buf, uint32_t first, uint32_t n) {
        float* dst = zs + (size_t)buf * CS * H;
        for (int p = threadIdx.x; p < pieces; p += blockDim.x) {
            const int r = p / (H / 4), k = (p % (H / 4)) * 4;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if ((uint32_t)r < n) {
                const uint4 it = __ldcg(reinterpret_cast<const uint4*>(&c.cell_sorted[first + r]));   // {out, l, r, height}
                if (it.x < c.frame_cap) v = ldcg4(c.dhp + (size_t)it.x * H + k);
                if (k == 0) s_rec[buf * CS + r] = it;
            }
            *reinterpret_cast<float4*>(dst + (size_t)r * H + k) = v;
        }
    };
    const uint32_t d0 = min(c.ctl->d_split, top);                     // (the grid-wide kernel ran depths 1 .. d0)
    // Only the dz rows of a depth depend on the depth above.  Everything else is known before the kernel starts and is
    // fetched ahead, off the chain of dependent waves: the records of a depth's first CS cells two depths ahead (ring in
    // shared memory), and what thread (cell ks, column jj) needs of its callee one depth ahead (registers).
    uint4* s_ring = s_rec + 2 * CS;                                    // [3][CS]; .x == 0xFFFFFFFF: no cell
    struct Callee { uint32_t child, child_l, child_tok; float4 dl0, dl1; float hv; };
    auto callee_of = [&](const uint4& rec, bool valid) {
        Callee q;
        q.child = 0xFFFFFFFFu; q.child_l = LEAF_MARK; q.child_tok = 0u;
        q.dl0 = make_float4(0.f, 0.f, 0.f, 0.f); q.dl1 = q.dl0; q.hv = 0.f;
        const uint32_t ch = col < H ? rec.y : rec.z;
        if (valid && col < K2 && rec.x < c.frame_cap && ch < c.frame_cap) {
            q.child = ch;
            q.child_l = c.op_l[ch]; q.child_tok = c.op_r[ch];
            q.dl0 = *reinterpret_cast<const float4*>(c.dlog + (size_t)ch * 8);
            q.dl1 = *reinterpret_cast<const float4*>(c.dlog + (size_t)ch * 8 + 4);
            q.hv = c.arena[(size_t)ch * H + cc];
        }
        return q;
    };
    auto first_record = [&](uint32_t d, uint32_t t) {                 // record t of depth d, or the empty record
        uint4 rec = make_uint4(0xFFFFFFFFu, 0u, 0u, 0u);
        if (d <= top) {
            const uint32_t b = min(ends[d - 1], c.work_cap), e = min(ends[d], c.work_cap);
            if (b + t < e) rec = __ldcg(reinterpret_cast<const uint4*>(&c.cell_sorted[b + t]));
        }
        return rec;
    };
    if (threadIdx.x < CS) {
        s_ring[((d0 + 1) % 3) * CS + threadIdx.x] = first_record(d0 + 1, threadIdx.x);
        s_ring[((d0 + 2) % 3) * CS + threadIdx.x] = first_record(d0 + 2, threadIdx.x);
    }
    __syncthreads();
    Callee ahead = callee_of(s_ring[((d0 + 1) % 3) * CS + (active ? ks : 0)], active);
    uint32_t begin = min(ends[d0], c.work_cap);
    for (uint32_t d = d0 + 1; d <= top; ++d) {
        const uint32_t end = min(ends[d], c.work_cap);
        uint4 rec_ahead = make_uint4(0xFFFFFFFFu, 0u, 0u, 0u);
        if (threadIdx.x < CS) rec_ahead = first_record(d + 2, threadIdx.x);             // lands while this depth runs
        int buf = 0;
        {   // first step: records from the ring, rows from the depth above
            const uint32_t n = min((uint32_t)CS, end - begin);
            for (int p = threadIdx.x; p < pieces; p += blockDim.x) {
                const int r = p / (H / 4), k = (p % (H / 4)) * 4;
                float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                const uint4 it = s_ring[(d % 3) * CS + r];
                if ((uint32_t)r < n && it.x < c.frame_cap) v = ldcg4(c.dhp + (size_t)it.x * H + k);
                if (k == 0) s_rec[r] = it;
                *reinterpret_cast<float4*>(zs + (size_t)r * H + k) = v;
            }
        }
        const Callee mine = ahead;
        ahead = callee_of(s_ring[((d + 1) % 3) * CS + (active ? ks : 0)], active && d + 1 <= top);   // used one depth on
        for (uint32_t first = begin; first < end; first += CS) {
            const uint32_t n = min((uint32_t)CS, end - first);
            __syncthreads();                                            // rows and records of this step are in place, `part` is free
            if (first + CS < end) stage(buf ^ 1, first + CS, min((uint32_t)CS, end - first - CS));
            // the callee that thread (cell ks, column jj) finishes after the contraction
            const Callee q = first == begin ? mine : callee_of(s_rec[buf * CS + (active ? ks : 0)], active && (uint32_t)ks < n);
            const bool fin = active && (uint32_t)ks < n && q.child < c.frame_cap;
            if (active) {
                float acc[CS];
#pragma unroll
                for (int qq = 0; qq < CS; ++qq) acc[qq] = 0.f;
                const float* z = zs + (size_t)buf * CS * H;
                for (int k = k_begin; k < k_end; k += 4) {
                    const float w0 = wres[(size_t)k * CPC + jj], w1 = wres[(size_t)(k + 1) * CPC + jj];
                    const float w2 = wres[(size_t)(k + 2) * CPC + jj], w3 = wres[(size_t)(k + 3) * CPC + jj];
#pragma unroll
                    for (int qq = 0; qq < CS; ++qq) {
                        const float4 zv = *reinterpret_cast<const float4*>(z + (size_t)qq * H + k);    // (one word for the whole warp)
                        acc[qq] = fmaf(zv.x, w0, fmaf(zv.y, w1, fmaf(zv.z, w2, fmaf(zv.w, w3, acc[qq]))));
                    }
                }
#pragma unroll
                for (int qq = 0; qq < CS; ++qq) part[((size_t)ks * CS + qq) * CPC + jj] = acc[qq];
            }
            __syncthreads();
            if (fin) {
                float t = 0.f;
#pragma unroll
                for (int qq = 0; qq < CS; ++qq) t += part[((size_t)qq * CS + ks) * CPC + jj];
                const float dl[MAX_CLASSES] = {q.dl0.x, q.dl0.y, q.dl0.z, q.dl0.w, q.dl1.x, q.dl1.y, q.dl1.z, q.dl1.w};
#pragma unroll
                for (int k = 0; k < MAX_CLASSES; ++k)
                    if (k < C) t = fmaf(__ldg(&c.W_s[k * H + cc]), dl[k], t);
                if (q.child_l == LEAF_MARK) {
                    if (q.child_tok < (uint32_t)c.V) atomicAdd(c.dE + (size_t)q.child_tok * c.D + cc, t);
                } else {
                    c.dhp[(size_t)q.child * H + cc] = t * (1.f - q.hv * q.hv);
                }
            }
            buf ^= 1;
        }
        begin = end;
        if (threadIdx.x < CS) s_ring[((d + 2) % 3) * CS + threadIdx.x] = rec_ahead;      // (slot of depth d - 1: no longer read)
        __syncthreads();
        cluster_sync_all();                                             // the rows of depth d + 1 are complete for the whole cluster
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) c.ctl->waves_backward += top - d0;      // (after the grid-wide kernel's count)
}

inline int bwd_cluster_cols_per_block(int H) { return H <= 64 ? 16 : H <= 128 ? 32 : H <= 256 ? 64 : 128; }
inline size_t bwd_cluster_smem_bytes(int H) {
    const int CPC = bwd_cluster_cols_per_block(H), CS = CPC <= 64 ? 8 : 4;
    return ((size_t)H * CPC + (size_t)2 * CS * H + (size_t)CS * CS * CPC) * sizeof(float) + 5 * CS * sizeof(uint4);
}

// ------------------------------------------- parameter gradients (post pass)
// out[m][n] = sum over the listed invocations t of A_t[m] * B_t[n]   (split over the list)
//   A_t = A + t * lda (M values: dz, or gate gradients)
//   mode 0: B_t = [h(l_t) ; h(r_t)]  (N = 2H)   -> dW
//   mode 1: B_t = E[tok_t]           (N = D)    -> dW_x (TreeLSTM leaves)
struct OuterArgs {
    const uint32_t* list;
    const uint32_t* count;
    const float* A;
    int lda, M, N, mode;
    float* out;
    int tiles_m, tiles_n;
    uint32_t chunk;
};

__global__ void __launch_bounds__(256) rdf_outer_kernel(const DevCtx c, const OuterArgs a) {
    if (c.ctl->status != 0) return;                    // an earlier kernel of this call failed: its lists and rows are not to be trusted
    __shared__ GemmSmem sm;
    const uint32_t n_items = *a.count;
    const int tile = blockIdx.x % (a.tiles_m * a.tiles_n), split = blockIdx.x / (a.tiles_m * a.tiles_n);
    const uint32_t t_begin = (uint32_t)split * a.chunk, t_end = min(n_items, t_begin + a.chunk);
    if (t_begin >= t_end) return;
    const int H = c.H, S = c.S;
    const int tm = tile / a.tiles_n, tn = tile % a.tiles_n;
    const int row0 = tm * TM, col0 = tn * TN;
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
    const int lk = threadIdx.x / 16, l4 = (threadIdx.x % 16) * 4;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
    for (uint32_t t0 = t_begin; t0 < t_end; t0 += TK) {
        float4 av = make_float4(0.f, 0.f, 0.f, 0.f), bv = av;
        if (t0 + lk < t_end) {
            const uint32_t t = a.list[t0 + lk];
            if (row0 + l4 < a.M) av = *reinterpret_cast<const float4*>(a.A + (size_t)t * a.lda + row0 + l4);
            const int col = col0 + l4;
            if (col < a.N) {
                if (a.mode == 0) {
                    const uint32_t src = col < H ? c.op_l[t] : c.op_r[t];
                    bv = *reinterpret_cast<const float4*>(c.arena + (size_t)src * S + (col < H ? col : col - H));
                } else {
                    bv = __ldg(reinterpret_cast<const float4*>(c.E + (size_t)c.op_r[t] * c.D + col));
                }
            }
        }
        __syncthreads();
        *reinterpret_cast<float4*>(&sm.As[lk][l4]) = av;
        *reinterpret_cast<float4*>(&sm.Bs[lk][l4]) = bv;
        __syncthreads();
        gemm_tile_step(sm, tx, ty, acc);
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int row = row0 + ty * 4 + i;
        if (row >= a.M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int col = col0 + tx * 4 + j;
            if (col < a.N) atomicAdd(&a.out[(size_t)row * a.N + col], acc[i][j]);
        }
    }
}

// out[g * H + u] = sum over the listed invocations of A_t[g * Hb + u]   (bias gradients; Hb = H for
// fp32 rows, the padded Hp for the bf16 operand rows)
__device__ __forceinline__ float as_float(float v) { return v; }
__device__ __forceinline__ float as_float(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename T>
__global__ void __launch_bounds__(256) rdf_colsum_kernel(const int32_t* status, const uint32_t* list, const uint32_t* count,
                                                         const T* A, int lda, int M, int H, int Hb, float* out) {
    if (*status != 0) return;                          // an earlier kernel of this call failed
    const uint32_t n = *count;
    const uint32_t per = (n + gridDim.x - 1) / gridDim.x;
    const uint32_t t0 = blockIdx.x * per, t1 = min(n, t0 + per);
    if (t0 >= t1) return;
    for (int j = threadIdx.x; j < M; j += blockDim.x) {
        const int col = (j / H) * Hb + j % H;
        float s = 0.f;
#pragma unroll 8
        for (uint32_t i = t0; i < t1; ++i) s += as_float(A[(size_t)(list ? list[i] : i) * lda + col]);
        atomicAdd(&out[j], s);
    }
}

// reproducible mode: one row of partial sums per block, the rows added up in block order
template <typename T>
__global__ void __launch_bounds__(256) rdf_colsum_partial_kernel(const int32_t* status, const uint32_t* list, const uint32_t* count,
                                                                 const T* A, int lda, int M, int H, int Hb, float* partial) {
    if (*status != 0) return;
    const uint32_t n = *count;
    const uint32_t per = (n + gridDim.x - 1) / gridDim.x;
    const uint32_t t0 = min(n, blockIdx.x * per), t1 = min(n, t0 + per);
    for (int j = threadIdx.x; j < M; j += blockDim.x) {
        const int col = (j / H) * Hb + j % H;
        float s = 0.f;
#pragma unroll 8
        for (uint32_t i = t0; i < t1; ++i) s += as_float(A[(size_t)(list ? list[i] : i) * lda + col]);
        partial[(size_t)blockIdx.x * M + j] = s;
    }
}
__global__ void __launch_bounds__(256) rdf_rows_reduce_kernel(const int32_t* status, const float* partial, int n_rows, int n, float* out) {
    if (*status != 0) return;
    const int q = blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= n) return;
    float t = 0.f;
    for (int r = 0; r < n_rows; ++r) t += partial[(size_t)r * n + q];
    out[q] = t;
}

// TreeLSTM: dE[tok_t] += W_x^T dg_t for every leaf t (dg_t = the 3H gate gradients)
__global__ void __launch_bounds__(256) rdf_de_lstm_kernel(const DevCtx c, int tiles_n) {
    if (c.ctl->status != 0) return;                    // an earlier kernel of this call failed: its lists and rows are not to be trusted
    __shared__ GemmSmem sm;
    const uint32_t n_items = c.ctl->all_leaves;
    const int D = c.D, Kdim = 3 * c.H;
    const int tiles_m = (n_items + TM - 1) / TM;
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
    const int arow_l = threadIdx.x / 4, ak = (threadIdx.x % 4) * 4;
    const int bk = threadIdx.x / 16, bn = (threadIdx.x % 16) * 4;
    for (int tile = blockIdx.x; tile < tiles_m * tiles_n; tile += gridDim.x) {
        const int tm = tile / tiles_n, tn = tile % tiles_n;
        const int row0 = tm * TM, col0 = tn * TN;
        const int arow = row0 + arow_l;
        const float* dg = arow < (int)n_items ? c.gates + (size_t)c.all_leaves[arow] * c.G : nullptr;
        float acc[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
        for (int k0 = 0; k0 < Kdim; k0 += TK) {
            float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
            if (dg && k0 + ak < Kdim) a = *reinterpret_cast<const float4*>(dg + k0 + ak);
            if (k0 + bk < Kdim && col0 + bn < D)
                b = __ldg(reinterpret_cast<const float4*>(c.W_x + (size_t)(k0 + bk) * D + col0 + bn));
            __syncthreads();
            sm.As[ak + 0][arow_l] = a.x; sm.As[ak + 1][arow_l] = a.y; sm.As[ak + 2][arow_l] = a.z; sm.As[ak + 3][arow_l] = a.w;
            *reinterpret_cast<float4*>(&sm.Bs[bk][bn]) = b;
            __syncthreads();
            gemm_tile_step(sm, tx, ty, acc);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int row = row0 + ty * 4 + i;
            if (row >= (int)n_items) continue;
            const uint32_t tok = c.op_r[c.all_leaves[row]];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int col = col0 + tx * 4 + j;
                if (col < D) atomicAdd(&c.dE[(size_t)tok * D + col], acc[i][j]);
            }
        }
    }
}

// --------------------------------------------------------------------- host
namespace {
OuterArgs outer_args(const uint32_t* list, const uint32_t* count, const float* A, int lda, int M, int N, int mode,
                     float* out, long long max_items, int grid) {
    OuterArgs a;
    a.list = list; a.count = count; a.A = A; a.lda = lda; a.M = M; a.N = N; a.mode = mode; a.out = out;
    a.tiles_m = (M + TM - 1) / TM;
    a.tiles_n = (N + TN - 1) / TN;
    const int tiles = a.tiles_m * a.tiles_n;
    const long long splits = std::max<long long>(1, std::min<long long>((max_items + 255) / 256, (4 * grid) / tiles + 1));
    uint32_t chunk = (uint32_t)((max_items + splits - 1) / splits);
    a.chunk = (chunk + TK - 1) / TK * TK;
    return a;
}
int outer_blocks(const OuterArgs& a, long long max_items) {
    return a.tiles_m * a.tiles_n * (int)((max_items + a.chunk - 1) / a.chunk);
}
}  // namespace

extern "C" int rdf_grad(rdf_graph* g, const rdf_batch* in, const rdf_params* params, rdf_outputs* out,
                        rdf_param_grads* grads, void* workspace, size_t workspace_bytes, void* stream_v) {
    int rc = rdf_check_common(g, in, params, out, workspace);
    if (rc != RDF_OK) return rc;
    if (!g->has_vector_ops || !g->has_loss) return RDF_ERR_UNSUPPORTED;
    if (!grads || !grads->dE || !grads->dW || !grads->db || !grads->dW_s || !grads->db_s) return RDF_ERR_BAD_ARG;
    if (g->has_lstm && (!grads->dW_x || !grads->db_x)) return RDF_ERR_BAD_ARG;
    if (!params->W_s || !params->b_s || !in->label || !out->loss) return RDF_ERR_BAD_ARG;
    if (params->n_classes < 1 || params->n_classes > MAX_CLASSES) return RDF_ERR_BAD_ARG;
    if (params->H > GRAD_MAX_H) return RDF_ERR_UNSUPPORTED;
    Layout L;
    rc = rdf_make_layout(g, in, params, 1, L);
    if (rc != RDF_OK) return rc;
    if (params->reproducible && !L.repro) return RDF_ERR_UNSUPPORTED;     // (only the tensor-core path has the ordered sums)
    if (workspace_bytes < L.total) return RDF_ERR_WORKSPACE_TOO_SMALL;
    ExecState* S = rdf_state_of(g);
    rc = rdf_prepare_device(g, S);
    if (rc != RDF_OK) return rc;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    char* ws = static_cast<char*>(workspace);
    DevCtx c;
    rdf_fill_ctx(g, in, params, out, ws, L, S, c);
    c.dE = grads->dE; c.dW = grads->dW; c.db = grads->db; c.dW_x = grads->dW_x; c.db_x = grads->db_x;
    c.dW_s = grads->dW_s; c.db_s = grads->db_s;
    const bool lstm = g->has_lstm;
    if (lstm) c.gates = reinterpret_cast<float*>(ws + L.gates);
    const int H = params->H, D = params->D;
    const int MW = lstm ? 5 * H : H;          // rows of W
    // gradients are sums: start from zero
    if (c.repro) {                         // the fixed-point sums start from zero; dE itself is written whole at the end
        CUDA_OK(cudaMemsetAsync(c.dE_fix, 0, (size_t)params->V * D * sizeof(long long), stream));
        CUDA_OK(cudaMemsetAsync(c.head_fix, 0, ((size_t)params->n_classes * (H + 1) + 1) * sizeof(long long), stream));
    } else CUDA_OK(cudaMemsetAsync(grads->dE, 0, (size_t)params->V * D * sizeof(float), stream));
    CUDA_OK(cudaMemsetAsync(grads->dW, 0, (size_t)MW * 2 * H * sizeof(float), stream));
    CUDA_OK(cudaMemsetAsync(grads->db, 0, (size_t)MW * sizeof(float), stream));
    CUDA_OK(cudaMemsetAsync(grads->dW_s, 0, (size_t)params->n_classes * H * sizeof(float), stream));
    CUDA_OK(cudaMemsetAsync(grads->db_s, 0, (size_t)params->n_classes * sizeof(float), stream));
    if (lstm) {
        CUDA_OK(cudaMemsetAsync(grads->dW_x, 0, (size_t)3 * H * D * sizeof(float), stream));
        CUDA_OK(cudaMemsetAsync(grads->db_x, 0, (size_t)3 * H * sizeof(float), stream));
    }
    rc = rdf_launch_forward(g, in, out, ws, L, S, c, stream);
    if (rc != RDF_OK) return rc;
    // loss head over every retained invocation
    const bool tc_rnn = c.use_tc && !lstm, tc_lstm = c.use_tc && lstm;
    if (tc_rnn) {                          // dz rows are read as 2D tiles by the gradient waves and by the weight gradient
        rc = encode_row_tiles(&c.tmap_dz128, c.dz_bf, c.cells_cap, (uint64_t)c.Hp, 128);
        if (rc == RDF_OK) rc = encode_row_tiles(&c.tmap_dz64, c.dz_bf, c.cells_cap, (uint64_t)c.Hp, 64);
        if (rc != RDF_OK) return rc;
    }
    {
        const int rowbytes = tc_rnn ? c.Hp * 2 : c.S * 4;
        const int fr = std::max(1, std::min(LH_MAX_ROWS, LH_SLAB_BYTES / rowbytes));
        const int smem = 2 * fr * rowbytes + params->n_classes * H * (int)sizeof(float);
        const int loss_blocks = std::min(4096, 2 * S->grid);
        if (c.repro) {
            RDF_KERNEL(S, rdf_loss_heads_exact_kernel<<<8 * S->grid, 256, 0, stream>>>(c));
            RDF_KERNEL(S, rdf_head_convert_kernel<<<(params->n_classes * (H + 1) + 1 + 255) / 256, 256, 0, stream>>>(c));
        } else if (c.use_tc) {             // bf16 states (TreeRNN and TreeLSTM): the h rows of arena_bf
            const int smem_mma = 2 * LM_ROWS * (c.Hp * 2 + 16);
            CUDA_OK(cudaFuncSetAttribute(rdf_loss_heads_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_mma));
            RDF_KERNEL(S, rdf_loss_heads_mma_kernel<<<loss_blocks, 256, smem_mma, stream>>>(c));
        } else {
            CUDA_OK(cudaFuncSetAttribute(rdf_loss_heads_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
            RDF_KERNEL(S, rdf_loss_heads_kernel<false><<<loss_blocks, 256, smem, stream>>>(c, fr, rowbytes));
        }
        if (!c.repro) RDF_KERNEL(S, rdf_loss_final_kernel<<<1, 256, 0, stream>>>(c, loss_blocks));
    }
    rdf_mark(S, 6, stream);
    // lists of the gradient pass (cells in frame order, the waves that made calls); the tensor-core forward pass made them already
    if (!c.use_tc) {
        rc = rdf_launch_lists(in, ws, L, S, c, stream);
        if (rc != RDF_OK) return rc;
    }
    rdf_mark(S, 7, stream);
    // gradient waves
    CUDA_OK(cudaGetLastError());
    void* args[] = {(void*)&c};
    if (c.use_tc) {
        CUDA_OK(cudaFuncSetAttribute(rdf_backward_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, L.tc_smem_bwd));
        RDF_KERNEL(S, CUDA_OK(cudaLaunchCooperativeKernel((void*)rdf_backward_kernel<true>, dim3(S->grid), dim3(TC_THREADS), args,
                                            (size_t)L.tc_smem_bwd, stream)));
    } else {
        // deep recursions: the cells grouped by (cluster of instances, call depth); the grid-wide kernel runs the wide depths,
        // the clusters the narrow ones after them (both leave at once when there is nothing for them to do)
        const bool clusters = c.n_groups > 1 && !c.lstm && H <= 512;
        if (clusters) {
            rc = rdf_launch_depth_groups(ws, L, S, c, stream);
            if (rc != RDF_OK) return rc;
        }
        if (c.lstm) {
            CUDA_OK(cudaFuncSetAttribute(rdf_backward_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 128 * THIN_RESIDENT_MAX_H));
            RDF_KERNEL(S, CUDA_OK(cudaLaunchCooperativeKernel((void*)rdf_backward_kernel<false>, dim3(S->grid), dim3(256), args,
                                                thin_resident_bytes(c.lstm, c.H), stream)));
        } else {
            // fp32 TreeRNN: as many blocks per SM as both of its persistent kernels take
            int per_sm = 0;
            CUDA_OK(cudaFuncSetAttribute(rdf_backward_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 128 * THIN_RESIDENT_MAX_H));
            CUDA_OK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, rdf_backward_kernel<false, true>, 256, 128 * THIN_RESIDENT_MAX_H));
            per_sm = std::max(1, std::min(per_sm, S->rnn32_per_sm));
            RDF_KERNEL(S, CUDA_OK(cudaLaunchCooperativeKernel((void*)rdf_backward_kernel<false, true>, dim3(S->grid * per_sm), dim3(256), args,
                                                thin_resident_bytes(0, c.H), stream)));
        }
        if (clusters) {
            cudaLaunchConfig_t cfg = {};
            cudaLaunchAttribute at[1];
            at[0].id = cudaLaunchAttributeClusterDimension;
            at[0].val.clusterDim.x = CLUSTER_CTAS; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
            cfg.gridDim = dim3(c.n_groups * CLUSTER_CTAS); cfg.blockDim = dim3(BWD_CLUSTER_THREADS);
            cfg.dynamicSmemBytes = bwd_cluster_smem_bytes(H); cfg.stream = stream;
            cfg.attrs = at; cfg.numAttrs = 1;
            const int smem = (int)cfg.dynamicSmemBytes;
            switch (bwd_cluster_cols_per_block(H)) {
                case 16:
                    CUDA_OK(cudaFuncSetAttribute(rdf_backward_cluster_kernel<16, 8>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
                    RDF_KERNEL(S, CUDA_OK(cudaLaunchKernelEx(&cfg, rdf_backward_cluster_kernel<16, 8>, c))); break;
                case 32:
                    CUDA_OK(cudaFuncSetAttribute(rdf_backward_cluster_kernel<32, 8>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
                    RDF_KERNEL(S, CUDA_OK(cudaLaunchKernelEx(&cfg, rdf_backward_cluster_kernel<32, 8>, c))); break;
                case 64:
                    CUDA_OK(cudaFuncSetAttribute(rdf_backward_cluster_kernel<64, 8>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
                    RDF_KERNEL(S, CUDA_OK(cudaLaunchKernelEx(&cfg, rdf_backward_cluster_kernel<64, 8>, c))); break;
                default:
                    CUDA_OK(cudaFuncSetAttribute(rdf_backward_cluster_kernel<128, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
                    RDF_KERNEL(S, CUDA_OK(cudaLaunchKernelEx(&cfg, rdf_backward_cluster_kernel<128, 4>, c))); break;
            }
        }
    }
    rdf_mark(S, 8, stream);
    // parameter gradients
    const long long max_cells = std::max<long long>(1, in->max_invocations / 2 + 1);
    const long long max_leaves = std::max<long long>(1, in->max_invocations);
    const float* dgA = lstm ? c.gates : c.dhp;
    const int lda = lstm ? c.G : H;
    if (c.use_tc) {
        // 256 x 256 tiles of the padded gradient, the invocations split over the remaining blocks
        CUDA_OK(cudaFuncSetAttribute(rdf_dw_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, DW_SMEM_BYTES));
        auto launch_dw = [&](DwArgs a, long long max_items) {
            a.tiles_n = (a.Np + DW_TILE - 1) / DW_TILE;
            a.n_tiles = ((a.Mp + DW_TILE - 1) / DW_TILE) * a.tiles_n;
            const long long stages = (max_items + DW_KT - 1) / DW_KT;
            a.splits = (int)std::max<long long>(1, std::min<long long>(std::min(S->grid, DW_BLOCKS_MAX) / a.n_tiles, stages));
            a.partial = c.repro ? c.dw_partial : nullptr;
            RDF_KERNEL(S, rdf_dw_tc_kernel<<<a.n_tiles * a.splits, 256, DW_SMEM_BYTES, stream>>>(c, a));
            if (c.repro) RDF_KERNEL(S, rdf_dw_reduce_kernel<<<2 * S->grid, 256, 0, stream>>>(c, a));   // the partial tiles, added up in split order
        };
        DwArgs a{};
        a.ops = c.cell_ops; a.count = &c.ctl->all_cells;
        a.A = tc_lstm ? c.dg_bf : c.dz_bf; a.lda = tc_lstm ? 5 * c.Hp : c.Hp; a.Mp = tc_lstm ? 5 * c.Hp : c.Hp;
        a.Np = 2 * c.Hp; a.mode = 0; a.out = grads->dW; a.ldo = 2 * H;
        a.a_tiles = tc_rnn ? 1 : 0;
        a.b_tiles = 1;                                              // [h_l ; h_r] of the listed cells: the operand rows
        a.bias_out = H < c.Hp ? grads->db : nullptr;                // db comes out of the same contraction
        launch_dw(a, max_cells);
        if (tc_lstm) {
            DwArgs x{};
            x.ops = c.leaf_ops; x.count = &c.ctl->all_leaves;
            x.A = c.dg_bf; x.lda = 5 * c.Hp; x.Mp = 3 * c.Hp; x.Np = c.Hp; x.mode = 1; x.out = grads->dW_x; x.ldo = D;
            x.bias_out = H < c.Hp ? grads->db_x : nullptr;
            launch_dw(x, max_leaves);
        }
    } else {
        OuterArgs aw = outer_args(c.all_cells, &c.ctl->all_cells, dgA, lda, MW, 2 * H, 0, grads->dW, max_cells, S->grid);
        RDF_KERNEL(S, rdf_outer_kernel<<<outer_blocks(aw, max_cells), 256, 0, stream>>>(c, aw));
        if (lstm) {
            OuterArgs ax = outer_args(c.all_leaves, &c.ctl->all_leaves, c.gates, c.G, 3 * H, D, 1, grads->dW_x, max_leaves, S->grid);
            RDF_KERNEL(S, rdf_outer_kernel<<<outer_blocks(ax, max_leaves), 256, 0, stream>>>(c, ax));
        }
    }
    rdf_mark(S, 9, stream);
    if (c.use_tc && H < c.Hp) {}        // (column H of the dW / dW_x contractions)
    else if (c.repro) {
        // column sums in two steps: a row of partial sums per block (in the buffer the weight gradient is done with), then
        // the rows added up in block order.  TreeRNN: dz rows are in all_cells order; TreeLSTM: bf16 gate-gradient rows.
        const int cs_blocks = std::min(8 * S->grid, (int)((size_t)DW_BLOCKS_MAX * 65536 / (5 * (size_t)H)));
        auto colsum = [&](const uint32_t* list, const uint32_t* count, const __nv_bfloat16* A, int lda_, int M, float* out_) {
            RDF_KERNEL(S, rdf_colsum_partial_kernel<__nv_bfloat16><<<cs_blocks, 256, 0, stream>>>(&c.ctl->status, list, count, A, lda_, M, H, c.Hp, c.dw_partial));
            RDF_KERNEL(S, rdf_rows_reduce_kernel<<<(M + 255) / 256, 256, 0, stream>>>(&c.ctl->status, c.dw_partial, cs_blocks, M, out_));
        };
        if (tc_rnn) colsum(nullptr, &c.ctl->all_cells, c.dz_bf, c.Hp, H, grads->db);
        else {
            colsum(c.all_cells, &c.ctl->all_cells, c.dg_bf, 5 * c.Hp, 5 * H, grads->db);
            colsum(c.all_leaves, &c.ctl->all_leaves, c.dg_bf, 5 * c.Hp, 3 * H, grads->db_x);
        }
    }
    else if (tc_rnn) RDF_KERNEL(S, rdf_colsum_kernel<__nv_bfloat16><<<8 * S->grid, 256, 0, stream>>>(&c.ctl->status, nullptr, &c.ctl->all_cells, c.dz_bf, c.Hp, H, H, c.Hp, grads->db));   // dz rows are in all_cells order
    else if (tc_lstm) {                 // the gate gradients exist as bf16 operand rows only
        RDF_KERNEL(S, rdf_colsum_kernel<__nv_bfloat16><<<8 * S->grid, 256, 0, stream>>>(&c.ctl->status, c.all_cells, &c.ctl->all_cells, c.dg_bf, 5 * c.Hp, 5 * H, H, c.Hp, grads->db));
        RDF_KERNEL(S, rdf_colsum_kernel<__nv_bfloat16><<<8 * S->grid, 256, 0, stream>>>(&c.ctl->status, c.all_leaves, &c.ctl->all_leaves, c.dg_bf, 5 * c.Hp, 3 * H, H, c.Hp, grads->db_x));
    } else {
        RDF_KERNEL(S, rdf_colsum_kernel<float><<<8 * S->grid, 256, 0, stream>>>(&c.ctl->status, c.all_cells, &c.ctl->all_cells, dgA, lda, MW, H, H, grads->db));
        if (lstm) RDF_KERNEL(S, rdf_colsum_kernel<float><<<8 * S->grid, 256, 0, stream>>>(&c.ctl->status, c.all_leaves, &c.ctl->all_leaves, c.gates, c.G, 3 * H, H, H, grads->db_x));
    }
    rdf_mark(S, 10, stream);      // (dW_s and db_s came from the loss-head pass)
    if (tc_lstm) {
        const int n_split = c.Hp / 64, de_smem = tc_smem_bytes(64, 3 * c.Hp, 0, 0, 5);
        CUDA_OK(cudaFuncSetAttribute(rdf_de_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, de_smem));
        RDF_KERNEL(S, rdf_de_tc_kernel<<<(S->grid / n_split) * n_split, TC_THREADS, de_smem, stream>>>(c));
    } else if (lstm) RDF_KERNEL(S, rdf_de_lstm_kernel<<<4 * S->grid, 256, 0, stream>>>(c, (D + TN - 1) / TN));
    // (TreeRNN: the leaves added their dh to dE during the gradient waves)
    if (c.repro) RDF_KERNEL(S, rdf_de_convert_kernel<<<8 * S->grid, 256, 0, stream>>>(c));
    rdf_mark(S, 11, stream);
    CUDA_OK(cudaGetLastError());
    return RDF_OK;
}
