// Lists over the frames of a call, formed once after the scheduler's waves and used by the tensor-core
// operator waves, the gradient waves and the weight gradient.
//
// Frame ids are handed out wave after wave (a frame records the scheduler wave its Call_i fired in), so
// the invocations of one call depth are one id range, and listing the cells in frame order puts the cells
// of every depth next to each other: `all_cells` / `cell_ops` in depth order, `cell_pos[frame]` = position.
// Small kernels: per-segment counts, scan of the counts, fill (with the end of every wave in the id space),
// the end of every wave in the cell list, and the compaction of the waves that made calls into
// wave_marks[k] = {first frame, one past the last frame, first cell, one past the last cell}, k = 0 ..
// ctl->n_depth_waves - 1.  Depth k's cells read the states of depth k + 1: the operator waves walk the list
// from its end, the gradient waves from its start.
// (Included by rdf_exec.cu only: it defines kernels.)
#pragma once
#include <cstring>

#include <cuda.h>              // CUtensorMap and the prototype of its encoder (the entry point is looked up at run time)

#include "rdf_exec.h"


__device__ __forceinline__ void list_flags(const DevCtx& c, uint32_t f0, uint32_t F, uint32_t (&l)[8], uint32_t (&r)[8],
                                           uint32_t& cells, uint32_t& leaves) {
    cells = leaves = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {                       // thread-contiguous: frames f0 + 8 tid + i
        const uint32_t f = f0 + threadIdx.x * 8 + i;
        l[i] = LEAF_MARK; r[i] = 0;
        if (f < F) {
            l[i] = c.op_l[f]; r[i] = c.op_r[f];
            if (l[i] != LEAF_MARK) ++cells; else ++leaves;
        }
    }
}

__global__ void __launch_bounds__(256) rdf_list_count_kernel(const DevCtx c, uint2* seg_counts) {
    if (c.ctl->status != 0) return;                    // an earlier kernel of this call failed: its lists and rows are not to be trusted
    __shared__ uint32_t wc[8], wl[8];
    const uint32_t F = min(c.ctl->frame_count.v, c.frame_cap), f0 = (uint32_t)c.B + blockIdx.x * LIST_SEG;
    uint32_t l[8], r[8], cells, leaves;
    list_flags(c, f0, F, l, r, cells, leaves);
    for (int o = 16; o > 0; o >>= 1) {
        cells += __shfl_xor_sync(0xffffffffu, cells, o);
        leaves += __shfl_xor_sync(0xffffffffu, leaves, o);
    }
    if (threadIdx.x % 32 == 0) { wc[threadIdx.x / 32] = cells; wl[threadIdx.x / 32] = leaves; }
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t a = 0, b = 0;
        for (int w = 0; w < 8; ++w) { a += wc[w]; b += wl[w]; }
        seg_counts[blockIdx.x] = make_uint2(a, b);
    }
    // the marks of this call's waves start empty (the fill kernel writes the ends of the waves that made calls)
    const uint32_t n_waves = min(c.ctl->waves, c.wave_cap);
    for (uint32_t w = blockIdx.x * blockDim.x + threadIdx.x; w < n_waves; w += gridDim.x * blockDim.x)
        c.wave_marks[w] = make_uint4(0u, 0u, 0u, 0u);
}

// one block: exclusive scan of the segment counts in place; totals to the control block
__global__ void __launch_bounds__(1024) rdf_list_scan_kernel(const DevCtx c, uint2* seg_counts, int n_seg) {
    if (c.ctl->status != 0) return;                    // an earlier kernel of this call failed: its lists and rows are not to be trusted
    __shared__ uint32_t wa[32], wb[32];
    const int per = (n_seg + 1023) / 1024, s0 = threadIdx.x * per, s1 = min(n_seg, s0 + per);
    const int lane = threadIdx.x % 32, warp = threadIdx.x / 32;
    uint32_t a = 0, b = 0;
    for (int i = s0; i < s1; ++i) { a += seg_counts[i].x; b += seg_counts[i].y; }
    uint32_t pa = a, pb = b;                            // inclusive scan over the threads
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t x = __shfl_up_sync(0xffffffffu, pa, o), y = __shfl_up_sync(0xffffffffu, pb, o);
        if (lane >= o) { pa += x; pb += y; }
    }
    if (lane == 31) { wa[warp] = pa; wb[warp] = pb; }
    __syncthreads();
    if (warp == 0) {
        uint32_t x = wa[lane], y = wb[lane];
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t u = __shfl_up_sync(0xffffffffu, x, o), v = __shfl_up_sync(0xffffffffu, y, o);
            if (lane >= o) { x += u; y += v; }
        }
        wa[lane] = x; wb[lane] = y;                     // inclusive over the warps
        if (lane == 31) { c.ctl->all_cells = x; c.ctl->all_leaves = y; }
    }
    __syncthreads();
    a = pa - a + (warp ? wa[warp - 1] : 0u);
    b = pb - b + (warp ? wb[warp - 1] : 0u);
    for (int i = s0; i < s1; ++i) {
        const uint2 v = seg_counts[i];
        seg_counts[i] = make_uint2(a, b);
        a += v.x; b += v.y;
    }
}

__global__ void __launch_bounds__(256) rdf_list_fill_kernel(const DevCtx c, const uint2* seg_base) {
    if (c.ctl->status != 0) return;                    // an earlier kernel of this call failed: its lists and rows are not to be trusted
    __shared__ uint32_t wc[8], wl[8];
    const uint32_t F = min(c.ctl->frame_count.v, c.frame_cap), f0 = (uint32_t)c.B + blockIdx.x * LIST_SEG;
    uint32_t l[8], r[8], cells, leaves;
    list_flags(c, f0, F, l, r, cells, leaves);
    // exclusive prefix of (cells, leaves) over the threads of the block
    uint32_t pc = cells, pl = leaves;
    const int lane = threadIdx.x % 32, warp = threadIdx.x / 32;
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t a = __shfl_up_sync(0xffffffffu, pc, o), b = __shfl_up_sync(0xffffffffu, pl, o);
        if (lane >= o) { pc += a; pl += b; }
    }
    if (lane == 31) { wc[warp] = pc; wl[warp] = pl; }
    __syncthreads();
    const uint2 sb = seg_base[blockIdx.x];
    uint32_t ic = sb.x + pc - cells, il = sb.y + pl - leaves;
    for (int w = 0; w < warp; ++w) { ic += wc[w]; il += wl[w]; }
    // ends of the waves in the id space: frame f is the last of its wave when the next frame belongs to a later one
    {
        const uint32_t fa = f0 + threadIdx.x * 8;
        uint32_t wv = fa < F ? c.frames[fa].label >> FRAME_WAVE_SHIFT : 0u;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint32_t f = fa + i;
            if (f >= F) break;
            const uint32_t wn = f + 1 < F ? c.frames[f + 1].label >> FRAME_WAVE_SHIFT : 0xFFFFFFFFu;
            if (wn != wv && wv < c.wave_cap) c.wave_marks[wv].x = f + 1;
            wv = wn;
        }
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const uint32_t f = f0 + threadIdx.x * 8 + i;
        if (f >= F) break;
        if (l[i] != LEAF_MARK) {
            c.all_cells[ic] = f;
            if (c.cell_ops) c.cell_ops[ic] = make_uint4(f, l[i], r[i], 1u);
            if (c.cell_pos) c.cell_pos[f] = ic;
            ++ic;
        } else {
            if (c.lstm) {
                c.all_leaves[il] = f;
                if (c.leaf_ops) c.leaf_ops[il] = make_uint4(f, r[i], 0u, 1u);      // r = token id of a leaf
            }
            ++il;
        }
    }
}

// marks[d].w = cells among the frames below marks[d].x: where wave d ends in all_cells.  One warp per wave.
__global__ void __launch_bounds__(256) rdf_list_ends_kernel(const DevCtx c, const uint2* seg_base) {
    if (c.ctl->status != 0) return;                    // an earlier kernel of this call failed: its lists and rows are not to be trusted
    const uint32_t lane = threadIdx.x % 32, n_warps = gridDim.x * blockDim.x / 32;
    const uint32_t n_waves = min(c.ctl->waves, c.wave_cap);
    const uint32_t F = min(c.ctl->frame_count.v, c.frame_cap), B = (uint32_t)c.B;
    for (uint32_t d = (blockIdx.x * blockDim.x + threadIdx.x) / 32; d < n_waves; d += n_warps) {
        const uint32_t f = max(B, min(c.wave_marks[d].x, F));
        const uint32_t seg = (f - B) / LIST_SEG, s0 = B + seg * LIST_SEG;      // (the segment array has one entry to spare)
        uint32_t cnt = 0;
        for (uint32_t g = s0 + lane; g < f; g += 32) cnt += c.op_l[g] != LEAF_MARK;
        for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
        if (lane == 0) c.wave_marks[d].w = seg_base[seg].x + cnt;
    }
    // the weight gradient reads dz and the operand rows in whole stages of 64 rows: the rows after the last cell are zero
    if (blockIdx.x == 0) {
        const uint32_t n = min(c.ctl->all_cells, c.cells_cap), n_end = min((n + 63u) & ~63u, c.cells_cap);
        if (c.dz_bf) {
            const uint32_t per_row = (uint32_t)c.Hp / 8;
            for (uint32_t q = threadIdx.x; q < (n_end - n) * per_row; q += blockDim.x)
                *reinterpret_cast<uint4*>(c.dz_bf + (size_t)(n + q / per_row) * c.Hp + (q % per_row) * 8) = make_uint4(0u, 0u, 0u, 0u);
        }
        if (c.z_bf) {
            const uint32_t per_row = (uint32_t)c.Hp / 4;
            for (uint32_t q = threadIdx.x; q < (n_end - n) * per_row; q += blockDim.x)
                *reinterpret_cast<uint4*>(c.z_bf + (size_t)(n + q / per_row) * 2 * c.Hp + (q % per_row) * 8) = make_uint4(0u, 0u, 0u, 0u);
        }
    }
}

// Where an invocation's state goes besides its own row: the operand row of the cell that called it
// (row = position of the caller in the cell list, half = the operand port that the call's Return_i feeds).
__global__ void __launch_bounds__(256) rdf_list_zdst_kernel(const DevCtx c) {
    if (c.ctl->status != 0 || !c.zdst) return;
    const uint32_t F = min(c.ctl->frame_count.v, c.frame_cap), B = (uint32_t)c.B;
    for (uint32_t f = B + blockIdx.x * blockDim.x + threadIdx.x; f < F; f += gridDim.x * blockDim.x) {
        const Frame fr = c.frames[f];
        const LabelInfo& L = c.labels[fr.label & FRAME_LABEL_MASK];
        uint32_t z = NO_ZDST;
        if (fr.parent >= B && fr.parent < F && L.k_kind == K_PORT && c.match[L.k_node].kind != MATCH_INT &&
            c.op_l[fr.parent] != LEAF_MARK)
            z = c.cell_pos[fr.parent] * 2u + (uint32_t)L.k_port;
        c.zdst[f] = z;
    }
}

// ---- reproducible mode: the cells of every depth in an order that depends on the input alone
// Frame ids are handed out in the order the scheduler's warps reach the frame counter, so the position of a cell
// among the cells of its depth differs from run to run, and with it the order of every sum over the cells.  Here the
// cells of a depth are re-ordered by the argument of their invocation (for the tree networks: the node index, which is
// unique), ties by their previous position.  A cell's rank is counted directly (every cell against the cells of its
// depth: about the square of the widest depth in comparisons, which is what this mode pays for).
// (leaves != 0: the same for the list of leaves -- the TreeLSTM's leaf projection sums over it; the leaves of a
// depth are the frames of the depth that are not cells, so their range in the leaf list follows from the two others)
__global__ void __launch_bounds__(256) rdf_canon_keys_kernel(const DevCtx c, int leaves) {
    if (c.ctl->status != 0) return;
    long long* key = reinterpret_cast<long long*>(c.rank_tmp);
    const uint32_t* list = leaves ? c.all_leaves : c.all_cells;
    const uint32_t n = leaves ? min(c.ctl->all_leaves, c.frame_cap) : min(c.ctl->all_cells, c.cells_cap);
    for (uint32_t p = blockIdx.x * blockDim.x + threadIdx.x; p < n; p += gridDim.x * blockDim.x)
        key[p] = c.frames[list[p]].arg;
}

__global__ void __launch_bounds__(256) rdf_canon_rank_kernel(const DevCtx c, int leaves) {
    if (c.ctl->status != 0) return;
    if (c.canon_hist && c.canon_hist[c.canon_cap] == 0u) return;          // (the linear-time pass did it)
    const long long* key = reinterpret_cast<const long long*>(c.rank_tmp);
    const uint32_t* list = leaves ? c.all_leaves : c.all_cells;
    const uint32_t n = leaves ? min(c.ctl->all_leaves, c.frame_cap) : min(c.ctl->all_cells, c.cells_cap);
    const uint32_t nw = min(c.ctl->n_depth_waves, c.wave_cap), B = (uint32_t)c.B;
    // first position of depth k in the list
    auto start_of = [&](uint32_t k) { const uint4 m = c.wave_marks[k]; return leaves ? m.x - B - m.z : m.z; };
    auto end_of = [&](uint32_t k) { const uint4 m = c.wave_marks[k]; return leaves ? m.y - B - m.w : m.w; };
    for (uint32_t p0 = blockIdx.x * blockDim.x; p0 < n; p0 += gridDim.x * blockDim.x) {
        const uint32_t p = p0 + threadIdx.x;
        if (p >= n) continue;
        // the depth that holds position p: the last one that starts at or before p
        uint32_t lo = 0, hi = nw;
        while (hi - lo > 1) {
            const uint32_t mid = (lo + hi) / 2;
            if (start_of(mid) <= p) lo = mid; else hi = mid;
        }
        const uint32_t c0 = start_of(lo), c1 = min(end_of(lo), n);
        const long long mine = key[p];
        uint32_t below = 0;
        for (uint32_t q = c0; q < c1; ++q) {
            const long long k = key[q];
            below += (k < mine) || (k == mine && q < p);
        }
        c.cell_pos[list[p]] = c0 + below;
    }
}

// ---- the same ranks in linear time, when the arguments are distinct node indices (the tree networks)
// A stable counting sort of the nodes, taken in index order, by the depth of the cell (leaf) they carry: node_info[a] =
// {list position + 1, depth + 1} is scattered from the list; the nodes are cut into segments of CANON_SEG, a warp per
// segment counts its nodes per depth, the counts are scanned down the segments per depth, and the warp walks its
// segment again, 32 nodes at a time in index order, handing out the places.  canon_hist[canon_cap] is a flag: set when
// an argument is no node index or occurs twice, or the table does not fit -- the quadratic kernel then does the work.
static const uint32_t CANON_SEG = 1024;

__global__ void __launch_bounds__(256) rdf_canon_node_kernel(const DevCtx c, int leaves) {
    if (c.ctl->status != 0) return;
    const uint32_t* list = leaves ? c.all_leaves : c.all_cells;
    const uint32_t n = leaves ? min(c.ctl->all_leaves, c.frame_cap) : min(c.ctl->all_cells, c.cells_cap);
    const uint32_t nw = min(c.ctl->n_depth_waves, c.wave_cap), B = (uint32_t)c.B;
    uint32_t* flag = c.canon_hist + c.canon_cap;
    const unsigned long long n_seg = ((unsigned long long)c.N + CANON_SEG - 1) / CANON_SEG;
    if (blockIdx.x == 0 && threadIdx.x == 0 && n_seg * nw > c.canon_cap) *flag = 1u;
    auto start_of = [&](uint32_t k) { const uint4 m = c.wave_marks[k]; return leaves ? m.x - B - m.z : m.z; };
    for (uint32_t p = blockIdx.x * blockDim.x + threadIdx.x; p < n; p += gridDim.x * blockDim.x) {
        uint32_t lo = 0, hi = nw;
        while (hi - lo > 1) {                                  // the depth that holds position p
            const uint32_t mid = (lo + hi) / 2;
            if (start_of(mid) <= p) lo = mid; else hi = mid;
        }
        const long long a = c.frames[list[p]].arg;
        if (a < 0 || a >= c.N) { *flag = 1u; continue; }
        const unsigned long long rec = (unsigned long long)(p + 1u) | ((unsigned long long)(lo + 1u) << 32);
        if (atomicExch(reinterpret_cast<unsigned long long*>(&c.node_info[a]), rec) != 0ull) *flag = 1u;
    }
}

// pass 0: count; pass 1: place (between them rdf_canon_colscan_kernel)
__global__ void __launch_bounds__(256) rdf_canon_sweep_kernel(const DevCtx c, int leaves, int place) {
    if (c.ctl->status != 0 || c.canon_hist[c.canon_cap] != 0u) return;
    const uint32_t* list = leaves ? c.all_leaves : c.all_cells;
    const uint32_t nw = min(c.ctl->n_depth_waves, c.wave_cap), B = (uint32_t)c.B, lane = threadIdx.x % 32;
    const uint32_t n_seg = (uint32_t)(((unsigned long long)c.N + CANON_SEG - 1) / CANON_SEG);
    for (uint32_t seg = (blockIdx.x * blockDim.x + threadIdx.x) / 32; seg < n_seg; seg += gridDim.x * blockDim.x / 32) {
        uint32_t* hist = c.canon_hist + (size_t)seg * nw;
        for (uint32_t j = 0; j < CANON_SEG; j += 32) {
            const long long a = (long long)seg * CANON_SEG + j + lane;
            const uint2 info = a < c.N ? c.node_info[a] : make_uint2(0u, 0u);
            const uint32_t k1 = info.y;                                    // depth + 1, 0: no entry of this list
            const unsigned peers = __match_any_sync(0xffffffffu, k1);
            if (k1 == 0u) continue;
            const uint32_t leader = __ffs(peers) - 1, cnt = __popc(peers);
            uint32_t base = 0;
            if (lane == leader) base = atomicAdd(&hist[k1 - 1], cnt);     // (pass 1: the places before this chunk)
            if (place) {
                base = __shfl_sync(peers, base, leader);
                const uint4 m = c.wave_marks[k1 - 1];
                const uint32_t c0 = leaves ? m.x - B - m.z : m.z;
                c.cell_pos[list[info.x - 1]] = c0 + base + __popc(peers & ((1u << lane) - 1u));
            }
        }
    }
}

// per depth, the counts of the segments become the number of entries in the segments before
__global__ void __launch_bounds__(256) rdf_canon_colscan_kernel(const DevCtx c) {
    if (c.ctl->status != 0 || c.canon_hist[c.canon_cap] != 0u) return;
    const uint32_t nw = min(c.ctl->n_depth_waves, c.wave_cap);
    const uint32_t n_seg = (uint32_t)(((unsigned long long)c.N + CANON_SEG - 1) / CANON_SEG);
    for (uint32_t k = blockIdx.x * blockDim.x + threadIdx.x; k < nw; k += gridDim.x * blockDim.x) {
        uint32_t run = 0;
        for (uint32_t seg = 0; seg < n_seg; ++seg) {
            const uint32_t t = c.canon_hist[(size_t)seg * nw + k];
            c.canon_hist[(size_t)seg * nw + k] = run;
            run += t;
        }
    }
}

// the lists rewritten in the new order (by frame: a cell or leaf knows its new position)
__global__ void __launch_bounds__(256) rdf_canon_scatter_kernel(const DevCtx c, int leaves) {
    if (c.ctl->status != 0) return;
    const uint32_t F = min(c.ctl->frame_count.v, c.frame_cap), B = (uint32_t)c.B;
    for (uint32_t f = B + blockIdx.x * blockDim.x + threadIdx.x; f < F; f += gridDim.x * blockDim.x) {
        const uint32_t l = c.op_l[f];
        if ((l == LEAF_MARK) != (leaves != 0)) continue;
        const uint32_t np = c.cell_pos[f];
        if (leaves) {
            c.all_leaves[np] = f;
            if (c.leaf_ops) c.leaf_ops[np] = make_uint4(f, c.op_r[f], 0u, 1u);
        } else {
            c.all_cells[np] = f;
            if (c.cell_ops) c.cell_ops[np] = make_uint4(f, l, c.op_r[f], 1u);
        }
    }
}

// The waves that made calls, compacted in place (one block): wave_marks[d] = {., end frame, ., end cell} for
// every scheduler wave d becomes wave_marks[k] = {first frame, end frame, first cell, end cell} for the k-th
// wave that has frames.  Ends grow with d, so "the end of the previous wave with frames" is a running maximum.
__global__ void __launch_bounds__(1024) rdf_wave_compact_kernel(const DevCtx c) {
    __shared__ uint32_t w_cnt[32], w_f[32], w_c[32];
    __shared__ uint32_t carry_cnt, carry_f, carry_c;
    if (c.ctl->status != 0) return;
    const uint32_t n_waves = min(c.ctl->waves, c.wave_cap), lane = threadIdx.x % 32, warp = threadIdx.x / 32;
    if (threadIdx.x == 0) { carry_cnt = 0; carry_f = (uint32_t)c.B; carry_c = 0; }
    __syncthreads();
    for (uint32_t d0 = 0; d0 < n_waves; d0 += 1024) {
        const uint32_t d = d0 + threadIdx.x;
        const uint4 m = d < n_waves ? c.wave_marks[d] : make_uint4(0u, 0u, 0u, 0u);
        const uint32_t has = m.x != 0u;
        uint32_t cnt = has, fe = m.x, ce = has ? m.w : 0u;                 // inclusive: count, max end frame, max end cell
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t a = __shfl_up_sync(0xffffffffu, cnt, o), b = __shfl_up_sync(0xffffffffu, fe, o),
                           e = __shfl_up_sync(0xffffffffu, ce, o);
            if ((int)lane >= o) { cnt += a; fe = max(fe, b); ce = max(ce, e); }
        }
        if (lane == 31) { w_cnt[warp] = cnt; w_f[warp] = fe; w_c[warp] = ce; }
        __syncthreads();
        if (warp == 0) {
            uint32_t a = w_cnt[lane], b = w_f[lane], e = w_c[lane];
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t x = __shfl_up_sync(0xffffffffu, a, o), y = __shfl_up_sync(0xffffffffu, b, o),
                               z = __shfl_up_sync(0xffffffffu, e, o);
                if ((int)lane >= o) { a += x; b = max(b, y); e = max(e, z); }
            }
            w_cnt[lane] = a; w_f[lane] = b; w_c[lane] = e;
        }
        __syncthreads();
        // exclusive values of this thread: what came before it in its warp, in the warps before, in the chunks before
        uint32_t p_cnt = __shfl_up_sync(0xffffffffu, cnt, 1), p_f = __shfl_up_sync(0xffffffffu, fe, 1),
                 p_c = __shfl_up_sync(0xffffffffu, ce, 1);
        if (lane == 0) { p_cnt = 0; p_f = 0; p_c = 0; }
        if (warp) { p_cnt += w_cnt[warp - 1]; p_f = max(p_f, w_f[warp - 1]); p_c = max(p_c, w_c[warp - 1]); }
        p_cnt += carry_cnt; p_f = max(p_f, carry_f); p_c = max(p_c, carry_c);
        __syncthreads();                                                   // every thread has read its wave and the carries
        if (has) c.wave_marks[p_cnt] = make_uint4(p_f, m.x, p_c, m.w);
        if (threadIdx.x == 1023) { carry_cnt = p_cnt + has; carry_f = max(p_f, m.x); carry_c = max(p_c, ce); }
        __syncthreads();
    }
    if (threadIdx.x == 0) c.ctl->n_depth_waves = carry_cnt;
}

// A row-major bf16 matrix [rows, cols] as a 2D tensor for tile copies: boxes of box_rows x 64 columns in the 128-byte swizzle.
typedef CUresult (*TensorMapEncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                           const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                           CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
int encode_row_tiles(TensorMap* out, void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    static_assert(sizeof(TensorMap) == sizeof(CUtensorMap), "tensor map size");
    static TensorMapEncodeTiledFn encode = nullptr;
    if (!encode) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess || !fn)
            return RDF_ERR_CUDA;
        encode = reinterpret_cast<TensorMapEncodeTiledFn>(fn);
    }
    const cuuint64_t dims[2] = {cols, rows}, strides[1] = {cols * 2};
    const cuuint32_t box[2] = {64, box_rows}, estr[2] = {1, 1};
    CUtensorMap m;
    if (encode(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return RDF_ERR_CUDA;
    memcpy(out, &m, sizeof(m));
    return RDF_OK;
}

