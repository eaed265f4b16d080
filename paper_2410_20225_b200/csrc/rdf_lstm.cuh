// Binary TreeLSTM, forward tiles (fp32 FMA).
//   cell: [i; f_l; f_r; o; u] = W [h_l; h_r] + b,  c = s(i) tanh(u) + s(f_l) c_l + s(f_r) c_r,  h = s(o) tanh(c)
//   leaf: [i; o; u] = W_x E[tok] + b_x,            c = s(i) tanh(u),                           h = s(o) tanh(c)
// One thread accumulates all NG gate pre-activations of its 4 x 4 (row, hidden unit) patch.
#pragma once
#include "rdf_exec.h"

__device__ __forceinline__ float sigmoid_f(float x) { return 1.f / (1.f + expf(-x)); }

template <int NG>
__device__ void lstm_forward_tiles(const DevCtx& c, LstmSmem& sm, uint32_t first, uint32_t n_items) {
    constexpr bool CELL = NG == 5;
    const int H = c.H, S = c.S, G = c.G;
    const int Kdim = CELL ? 2 * H : c.D;
    const int split = CELL ? H : c.D;          // k < split comes from the first source row
    const float* Wm = CELL ? c.W : c.W_x;
    const float* bias = CELL ? c.b : c.b_x;
    const int tiles_m = (n_items + TM - 1) / TM, tiles_n = (H + TN - 1) / TN;
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
    const int lrow = threadIdx.x / 4, lk = (threadIdx.x % 4) * 4;
    for (int tile = blockIdx.x; tile < tiles_m * tiles_n; tile += gridDim.x) {
        const int tm = tile / tiles_n, tn = tile % tiles_n;
        const int row0 = tm * TM, col0 = tn * TN;
        const int arow = row0 + lrow;
        const float *xl = nullptr, *xr = nullptr;
        if (arow < (int)n_items) {
            if constexpr (CELL) {
                const uint4 it = __ldcg(reinterpret_cast<const uint4*>(&c.cell_items[first + arow]));   // {out, l, r, -}
                xl = c.arena + (size_t)it.y * S;
                xr = c.arena + (size_t)it.z * S;
            } else {
                const uint2 it = __ldcg(reinterpret_cast<const uint2*>(&c.leaf_items[arow]));  // {slot, tok}
                xl = c.E + (size_t)it.y * c.D;
            }
        }
        const int bcol = col0 + lrow;
        float acc[NG][4][4];
#pragma unroll
        for (int g = 0; g < NG; ++g)
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[g][i][j] = 0.f;
        for (int k0 = 0; k0 < Kdim; k0 += TK) {
            const int k = k0 + lk;
            float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
            float4 b[NG];
            if (xl && k < Kdim) a = k < split ? ldcg4(xl + k) : ldcg4(xr + (k - split));
#pragma unroll
            for (int g = 0; g < NG; ++g) {
                b[g] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (bcol < H && k < Kdim)
                    b[g] = __ldg(reinterpret_cast<const float4*>(Wm + (size_t)(g * H + bcol) * Kdim + k));
            }
            __syncthreads();
            sm.As[lk + 0][lrow] = a.x; sm.As[lk + 1][lrow] = a.y; sm.As[lk + 2][lrow] = a.z; sm.As[lk + 3][lrow] = a.w;
#pragma unroll
            for (int g = 0; g < NG; ++g) {
                sm.Bs[g][lk + 0][lrow] = b[g].x; sm.Bs[g][lk + 1][lrow] = b[g].y;
                sm.Bs[g][lk + 2][lrow] = b[g].z; sm.Bs[g][lk + 3][lrow] = b[g].w;
            }
            __syncthreads();
#pragma unroll
            for (int kk = 0; kk < TK; ++kk) {
                const float4 av = *reinterpret_cast<const float4*>(&sm.As[kk][ty * 4]);
                const float aa[4] = {av.x, av.y, av.z, av.w};
#pragma unroll
                for (int g = 0; g < NG; ++g) {
                    const float4 bv = *reinterpret_cast<const float4*>(&sm.Bs[g][kk][tx * 4]);
                    const float bb[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
                    for (int i = 0; i < 4; ++i)
#pragma unroll
                        for (int j = 0; j < 4; ++j) acc[g][i][j] = fmaf(aa[i], bb[j], acc[g][i][j]);
                }
            }
        }
        const int col = col0 + tx * 4;
        if (col < H) {
            float bz[NG][4];
#pragma unroll
            for (int g = 0; g < NG; ++g) {
                const float4 t = __ldg(reinterpret_cast<const float4*>(bias + g * H + col));
                bz[g][0] = t.x; bz[g][1] = t.y; bz[g][2] = t.z; bz[g][3] = t.w;
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int row = row0 + ty * 4 + i;
                if (row >= (int)n_items) continue;
                float hv[4], cv[4], gv[NG][4];
                uint32_t out;
                if constexpr (CELL) {
                    const uint4 it = __ldcg(reinterpret_cast<const uint4*>(&c.cell_items[first + row]));
                    out = it.x;
                    const float4 cl4 = ldcg4(c.arena + (size_t)it.y * S + H + col);
                    const float4 cr4 = ldcg4(c.arena + (size_t)it.z * S + H + col);
                    const float cl[4] = {cl4.x, cl4.y, cl4.z, cl4.w}, cr[4] = {cr4.x, cr4.y, cr4.z, cr4.w};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const float gi = sigmoid_f(acc[0][i][j] + bz[0][j]);
                        const float fl = sigmoid_f(acc[1][i][j] + bz[1][j]);
                        const float fr = sigmoid_f(acc[2][i][j] + bz[2][j]);
                        const float go = sigmoid_f(acc[3][i][j] + bz[3][j]);
                        const float gu = tanhf(acc[4][i][j] + bz[4][j]);
                        cv[j] = gi * gu + fl * cl[j] + fr * cr[j];
                        hv[j] = go * tanhf(cv[j]);
                        gv[0][j] = gi; gv[1][j] = fl; gv[2][j] = fr; gv[3][j] = go; gv[4][j] = gu;
                    }
                } else {
                    out = __ldcg(&c.leaf_items[row].slot);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const float gi = sigmoid_f(acc[0][i][j] + bz[0][j]);
                        const float go = sigmoid_f(acc[1][i][j] + bz[1][j]);
                        const float gu = tanhf(acc[2][i][j] + bz[2][j]);
                        cv[j] = gi * gu;
                        hv[j] = go * tanhf(cv[j]);
                        gv[0][j] = gi; gv[1][j] = go; gv[2][j] = gu;
                    }
                }
                float* st = c.arena + (size_t)out * S;
                *reinterpret_cast<float4*>(st + col) = make_float4(hv[0], hv[1], hv[2], hv[3]);
                *reinterpret_cast<float4*>(st + H + col) = make_float4(cv[0], cv[1], cv[2], cv[3]);
                if (c.gates) {
                    float* gt = c.gates + (size_t)out * G;
#pragma unroll
                    for (int g = 0; g < NG; ++g)
                        *reinterpret_cast<float4*>(gt + g * H + col) = make_float4(gv[g][0], gv[g][1], gv[g][2], gv[g][3]);
                }
            }
        }
    }
}
