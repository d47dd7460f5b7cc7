// Tiled FP32 scoring kernel for heads of any size.
//
// A tile holds up to 64 requests of one (instance, application) group, so the logits of the tile are a
// small GEMM  Z[64 x C] = X[64 x D] * W_a[D x C].  Classes are swept in chunks of 64 with an online
// softmax (running max, running sum, running sum of exp * recall), so neither the logits nor the
// posterior ever leave the SM: only acc[request][model] (Eq. 9) and v = 1 + Var (Eq. 12) are written.
#pragma once

#include "sp_common.cuh"
#include "sp_group.cuh"

namespace sp {

constexpr int kTiledThreads = 256;
constexpr int kTiledCols = 64;    // classes per chunk
constexpr int kTiledK = 16;       // feature-dimension slice per step

template <bool BF16>
__global__ void __launch_bounds__(kTiledThreads)
k_score_tiled(DevProfiles P, DevTable tb, const int32_t *__restrict__ tiled_start, float *__restrict__ acc_out,
              const int *__restrict__ flags) {
    __shared__ __align__(16) float Xs[kTiledK][kTiledRows + 4];   // k-major: a thread reads 4 consecutive rows
    __shared__ __align__(16) float Ws[kTiledK][kTiledCols];
    __shared__ __align__(16) float Rs[kMaxModelsPerApp][kTiledCols];
    __shared__ float Bs[kTiledCols];
    __shared__ int64_t s_req[kTiledRows];
    __shared__ int s_key, s_rows;

    const int tid = threadIdx.x;
    const int A = P.A, C = P.C, D = P.D;
    const int n_keys = P.I * A;
    if (tid == 0) {
        const int t = blockIdx.x;
        if (flags[1] || t >= tiled_start[n_keys]) s_key = -1;
        else {
            int lo = 0, hi = n_keys;
            while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (tiled_start[mid] <= t) lo = mid; else hi = mid; }
            s_key = lo;
        }
    }
    __syncthreads();
    const int key = s_key;
    if (key < 0) return;
    const int inst = key / A, a = key - inst * A;
    {
        const int64_t g0 = tb.gstart[key], g1 = tb.gstart[key + 1];
        const int64_t first = g0 + (int64_t)(blockIdx.x - tiled_start[key]) * kTiledRows;
        const int rows = (int)((g1 - first) < kTiledRows ? (g1 - first) : kTiledRows);
        if (tid < kTiledRows) s_req[tid] = tb.perm[first + (tid < rows ? tid : 0)];
        if (tid == 0) s_rows = rows;
    }
    __syncthreads();
    const int rows = s_rows;
    const int m0 = P.mfirst[a], M = P.mfirst[a + 1] - m0;
    const int64_t head = (int64_t)inst * A + a;
    const int ty = tid >> 4, tx = tid & 15;          // thread owns rows ty*4..+3, columns tx*4..+3 of a chunk

    float run_m[4], run_s[4], accA[4][kMaxModelsPerApp];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        run_m[i] = -INFINITY; run_s[i] = 0.f;
#pragma unroll
        for (int j = 0; j < kMaxModelsPerApp; ++j) accA[i][j] = 0.f;
    }

    // loader roles: X: row = tid/4, 4 consecutive k;  W: k = tid/16, 4 consecutive columns
    const int xr = tid >> 2, xk = (tid & 3) * 4;
    const int wk = tid >> 4, wc = (tid & 15) * 4;
    const int64_t xrow = s_req[xr] * (int64_t)D;

    for (int c0 = 0; c0 < C; c0 += kTiledCols) {
        float z[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) z[i][j] = 0.f;

        for (int k0 = 0; k0 < D; k0 += kTiledK) {
            float xv[4], wv[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int k = k0 + xk + i;
                float v = 0.f;
                if (k < D) v = BF16 ? bf16_bits_to_float(((const unsigned short *)tb.feats)[xrow + k])
                                    : ((const float *)tb.feats)[xrow + k];
                xv[i] = v;
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int k = k0 + wk, c = c0 + wc + j;
                float v = 0.f;
                if (k < D && c < C) {
                    const int64_t idx = (head * D + k) * C + c;
                    v = BF16 ? bf16_bits_to_float(((const unsigned short *)P.W)[idx]) : ((const float *)P.W)[idx];
                }
                wv[j] = v;
            }
            __syncthreads();                           // previous slice fully consumed
#pragma unroll
            for (int i = 0; i < 4; ++i) Xs[xk + i][xr] = xv[i];
            *reinterpret_cast<float4 *>(&Ws[wk][wc]) = make_float4(wv[0], wv[1], wv[2], wv[3]);
            __syncthreads();
#pragma unroll
            for (int k = 0; k < kTiledK; ++k) {
                const float4 xa = *reinterpret_cast<const float4 *>(&Xs[k][ty * 4]);
                const float4 wb = *reinterpret_cast<const float4 *>(&Ws[k][tx * 4]);
                const float xr4[4] = {xa.x, xa.y, xa.z, xa.w}, wc4[4] = {wb.x, wb.y, wb.z, wb.w};
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int j = 0; j < 4; ++j) z[i][j] = fmaf(xr4[i], wc4[j], z[i][j]);
            }
        }
        // ---- bias and recall columns of this chunk
        __syncthreads();
        if (tid < kTiledCols) {
            const int c = c0 + tid;
            Bs[tid] = c < C ? P.bias[head * C + c] : -INFINITY;
        }
        for (int k = tid; k < kMaxModelsPerApp * kTiledCols; k += kTiledThreads) {
            const int j = k / kTiledCols, cc = k - j * kTiledCols, c = c0 + cc;
            Rs[j][cc] = (j < M && c < C) ? P.recall[((int64_t)inst * P.sumM + m0 + j) * C + c] : 0.f;
        }
        __syncthreads();
        // ---- online softmax update; the 16 threads of a row are 16 consecutive lanes
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float cm = -INFINITY;
#pragma unroll
            for (int j = 0; j < 4; ++j) { z[i][j] += Bs[tx * 4 + j]; cm = fmaxf(cm, z[i][j]); }
#pragma unroll
            for (int o = 8; o >= 1; o >>= 1) cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, o));
            const float nm = fmaxf(run_m[i], cm);
            const float scale = run_m[i] == -INFINITY ? 0.f : expf(run_m[i] - nm);
            float ps = 0.f, p[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) { p[j] = nm == -INFINITY ? 0.f : expf(z[i][j] - nm); ps += p[j]; }
            run_s[i] = run_s[i] * scale + ps;          // per-thread partial of the row sum
            run_m[i] = nm;
#pragma unroll
            for (int jm = 0; jm < kMaxModelsPerApp; ++jm) {
                if (jm < M) {
                    const float4 r = *reinterpret_cast<const float4 *>(&Rs[jm][tx * 4]);
                    float t = accA[i][jm] * scale;
                    t = fmaf(p[0], r.x, t); t = fmaf(p[1], r.y, t); t = fmaf(p[2], r.z, t); t = fmaf(p[3], r.w, t);
                    accA[i][jm] = t;
                }
            }
        }
    }
    // ---- combine the 16 partials of each row, finish Eq. 9 / Eq. 12, write
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float s = run_s[i];
#pragma unroll
        for (int o = 8; o >= 1; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        const float inv = 1.f / s;
        float mean = 0.f, accv[kMaxModelsPerApp];
#pragma unroll
        for (int jm = 0; jm < kMaxModelsPerApp; ++jm) {
            float t = accA[i][jm];
#pragma unroll
            for (int o = 8; o >= 1; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
            t *= inv;
            if (jm < M) {
                if (P.prior)
                    t = (P.prior_dot[(int64_t)inst * P.sumM + m0 + jm] + P.kappa * t) / (P.prior_sum[head] + P.kappa);
                mean += t;
            } else t = 0.f;
            accv[jm] = t;
        }
        mean /= (float)M;
        float var = 0.f;
#pragma unroll
        for (int jm = 0; jm < kMaxModelsPerApp; ++jm)
            if (jm < M) var = fmaf(accv[jm] - mean, accv[jm] - mean, var);
        const int r = ty * 4 + i;
        if (r < rows) {
            const int64_t req = s_req[r];
            // the 16 lanes of the row share the stores
            for (int jm = tx; jm < P.Mmax; jm += 16) {
                float val = 0.f;
#pragma unroll
                for (int q = 0; q < kMaxModelsPerApp; ++q) if (q == jm) val = accv[q];
                tb.acc32[req * P.Mmax + jm] = val;
                if (acc_out) acc_out[req * P.Mmax + jm] = val;
            }
            if (tx == 0) tb.v32[req] = 1.f + var / (float)M;
        }
    }
}

}  // namespace sp
