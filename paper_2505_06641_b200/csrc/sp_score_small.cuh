// Scoring kernel for small heads (C <= 64 labels, every head of an instance fits in shared memory).
//
// Per request (Section 4.1 + Eq. 9 + Eq. 12 of the paper):
//   z = x W_a + b_a;  p = softmax(z);  theta = Dirichlet posterior mean;  acc_j = sum_c theta_c recall_j(c);
//   v = 1 + population variance_j(acc_j).
// The kernel is bound by reading x from HBM once, so the layout serves that: a tile of consecutive
// requests of one instance is staged in shared memory with 16-byte async copies, rows are placed in
// application order so that a warp works on requests that share one head (its weights are then
// broadcast reads), and each lane keeps RT x CT logits in registers (2 requests x half of the classes).
#pragma once

#include "sp_common.cuh"
#include "sp_group.cuh"

namespace sp {

constexpr int kSmallThreads = 256;
constexpr int kSmallWarps = kSmallThreads / 32;

__device__ __forceinline__ void cp_async16(void *smem, const void *gmem) {
    const unsigned s = (unsigned)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(s), "l"(gmem));
}
__device__ __forceinline__ void cp_async_commit_wait_all() {
    asm volatile("cp.async.commit_group;\ncp.async.wait_group 0;\n" ::: "memory");
}

struct SmallSmem {   // offsets in floats into dynamic shared memory
    int w, bias, recall, x, end;
    __host__ __device__ SmallSmem(int A, int D, int sumM, int ctp) {
        w = 0;
        bias = w + A * D * 2 * ctp;
        recall = bias + A * 2 * ctp;
        x = recall + sumM * 2 * ctp;
        x = (x + 3) & ~3;
        end = x + kSmallRows * (D + 4);
    }
};

template <int CT>
__device__ __forceinline__ void load_half_row(float (&w)[CT], const float *p) {
#pragma unroll
    for (int q = 0; q + 4 <= CT; q += 4) {
        const float4 t = *reinterpret_cast<const float4 *>(p + q);
        w[q] = t.x; w[q + 1] = t.y; w[q + 2] = t.z; w[q + 3] = t.w;
    }
    if (CT % 4 >= 2) {
        const float2 t = *reinterpret_cast<const float2 *>(p + (CT & ~3));
        w[CT & ~3] = t.x; w[(CT & ~3) + 1] = t.y;
    }
    if (CT % 2) w[CT - 1] = p[CT - 1];
}

// Tile descriptors: tile t -> (instance, first request relative to the instance, rows, first request in the table),
// instance = -1 past the end.  The last component is only meaningful below 2^31 requests (the tensor-core kernel,
// whose TMA coordinates are 32-bit, is the one that reads it).
__global__ void k_small_tiles(DevProfiles P, DevTable tb, const int32_t *__restrict__ small_start, int n_tiles,
                              int4 *__restrict__ desc, const int *__restrict__ flags) {
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= n_tiles) return;
    int4 d = make_int4(-1, 0, 0, 0);
    if (!flags[1] && t < small_start[P.I]) {
        int lo = 0, hi = P.I;                 // instance with small_start[inst] <= t < small_start[inst + 1]
        while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (small_start[mid] <= t) lo = mid; else hi = mid; }
        const int64_t i0 = tb.gstart[(int64_t)lo * P.A], i1 = tb.gstart[(int64_t)(lo + 1) * P.A];
        const int64_t r0 = (int64_t)(t - small_start[lo]) * kSmallRows;
        d = make_int4(lo, (int)r0, (int)((i1 - i0 - r0) < kSmallRows ? (i1 - i0 - r0) : kSmallRows), (int)(i0 + r0));
    }
    desc[t] = d;
}

// Copies `nrows` rows of C floats from global memory into the two-halves layout [row][2][CTP] used by the
// kernel below (lane half h owns labels h*CT .. h*CT+CT-1); positions without a label get `fill`.
// Loads are issued in batches so that one global-memory latency covers many elements.
template <int CT>
__device__ __forceinline__ void stage_halves(float *__restrict__ dst, const float *__restrict__ src, int nrows, int C,
                                             float fill) {
    constexpr int CTP = (CT + 3) & ~3;
    constexpr int U = 8;
    const int tid = threadIdx.x;
    if ((C & 3) == 0 && (((uintptr_t)src) & 15) == 0) {
        // labels come in aligned groups of four: vector loads, scalar scatter; padding written separately
        const int c4 = C >> 2, total = nrows * c4;
        for (int q0 = tid; q0 < total; q0 += kSmallThreads * U) {
            float4 v[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int q = q0 + u * kSmallThreads;
                v[u] = q < total ? reinterpret_cast<const float4 *>(src)[q] : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int q = q0 + u * kSmallThreads;
                if (q < total) {
                    const int row = q / c4, c = (q - row * c4) * 4;
                    const float e[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const int cc = c + k, h = cc >= CT ? 1 : 0;
                        dst[(row * 2 + h) * CTP + cc - h * CT] = e[k];
                    }
                }
            }
        }
        const int lab1 = C - CT > 0 ? C - CT : 0;         // labels in the second half
        const int lab0 = C < CT ? C : CT;
        const int pad0 = CTP - lab0, pad1 = CTP - lab1, pads = pad0 + pad1;
        for (int k = tid; k < nrows * pads; k += kSmallThreads) {
            const int row = k / pads, r = k - row * pads;
            if (r < pad0) dst[(row * 2) * CTP + lab0 + r] = fill;
            else dst[(row * 2 + 1) * CTP + lab1 + (r - pad0)] = fill;
        }
    } else {
        const int total = nrows * 2 * CTP;
        for (int k0 = tid; k0 < total; k0 += kSmallThreads * U) {
            float v[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int k = k0 + u * kSmallThreads;
                const int c2 = k % (2 * CTP), row = k / (2 * CTP);
                const int h = c2 / CTP, cc = c2 - h * CTP, c = h * CT + cc;
                v[u] = (k < total && cc < CT && c < C) ? src[(int64_t)row * C + c] : fill;
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int k = k0 + u * kSmallThreads;
                if (k < total) dst[k] = v[u];
            }
        }
    }
}

// CT = labels per lane (two lanes share a request, so C <= 2*CT).
template <int CT>
__global__ void __launch_bounds__(kSmallThreads, 2)
k_score_small(DevProfiles P, DevTable tb, const int4 *__restrict__ tiles, float *__restrict__ acc_out) {
    constexpr int CTP = (CT + 3) & ~3;
    extern __shared__ __align__(16) float smem[];
    __shared__ int s_cnt[kMaxApps], s_first[kMaxApps + 1], s_unit0[kMaxApps + 1];
    __shared__ short s_phys[kSmallRows];          // request of the tile -> row in shared memory
    __shared__ short s_local[kSmallRows];         // row in shared memory -> request of the tile

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int A = P.A, C = P.C, D = P.D;
    const SmallSmem L(A, D, P.sumM, CTP);

    const int4 desc = tiles[blockIdx.x];
    const int inst = desc.x;
    if (inst < 0) return;
    const int64_t row0 = tb.gstart[(int64_t)inst * A] + desc.y;
    const int rows = desc.z;
    if (tid < kMaxApps) s_cnt[tid] = 0;
    __syncthreads();

    // ---- applications of the tile's requests -> rows in application order
    int my_app = 0, my_rank = 0;
    if (tid < rows) {
        my_app = tb.app[row0 + tid];
        my_rank = atomicAdd(&s_cnt[my_app], 1);
    }
    __syncthreads();
    if (tid == 0) {
        int f = 0, u = 0;
        for (int a = 0; a < A; ++a) {
            s_first[a] = f; s_unit0[a] = u;
            f += s_cnt[a]; u += (s_cnt[a] + 31) >> 5;
        }
        s_first[A] = f; s_unit0[A] = u;
    }
    __syncthreads();
    if (tid < rows) {
        const int phys = s_first[my_app] + my_rank;
        s_phys[tid] = (short)phys;
        s_local[phys] = (short)tid;
    }
    __syncthreads();

    // ---- stage the feature rows (async 16-byte copies) and this instance's heads and profiles
    {
        const float *feats = (const float *)tb.feats;
        float *xs = smem + L.x;
        const int chunks = D >> 2;
        for (int k = tid; k < rows * chunks; k += kSmallThreads) {
            const int r = k / chunks, q = k - r * chunks;
            cp_async16(xs + s_phys[r] * (D + 4) + q * 4, feats + (row0 + r) * D + q * 4);
        }
        stage_halves<CT>(smem + L.w, (const float *)P.W + (int64_t)inst * A * D * C, A * D, C, 0.f);
        stage_halves<CT>(smem + L.bias, P.bias + (int64_t)inst * A * C, A, C, -INFINITY);
        stage_halves<CT>(smem + L.recall, P.recall + (int64_t)inst * P.sumM * C, P.sumM, C, 0.f);
        cp_async_commit_wait_all();
    }
    __syncthreads();

    // ---- units of 32 same-application rows; lane = (row slot 0..15, class half); 2 rows per lane
    const int n_units = s_unit0[A];
    const int rslot = lane & 15, h = lane >> 4;
    for (int u = warp; u < n_units; u += kSmallWarps) {
        int a = 0;
        while (u >= s_unit0[a + 1]) ++a;
        const int base = s_first[a] + (u - s_unit0[a]) * 32;
        const int lim = s_first[a + 1];
        const int p0 = base + rslot, p1 = base + 16 + rslot;
        const bool ok0 = p0 < lim, ok1 = p1 < lim;
        const float *x0 = smem + L.x + (ok0 ? p0 : 0) * (D + 4);
        const float *x1 = smem + L.x + (ok1 ? p1 : 0) * (D + 4);
        const float *wrow = smem + L.w + (a * D * 2 + h) * CTP;
        float z0[CT], z1[CT];
        load_half_row<CT>(z0, smem + L.bias + (a * 2 + h) * CTP);
#pragma unroll
        for (int c = 0; c < CT; ++c) z1[c] = z0[c];
        for (int d = 0; d < D; d += 4) {
            const float4 a0 = *reinterpret_cast<const float4 *>(x0 + d);
            const float4 a1 = *reinterpret_cast<const float4 *>(x1 + d);
            const float xa[4] = {a0.x, a0.y, a0.z, a0.w}, xb[4] = {a1.x, a1.y, a1.z, a1.w};
#pragma unroll
            for (int dd = 0; dd < 4; ++dd) {
                float w[CT];
                load_half_row<CT>(w, wrow + (d + dd) * 2 * CTP);
#pragma unroll
                for (int c = 0; c < CT; ++c) {
                    z0[c] = fmaf(xa[dd], w[c], z0[c]);
                    z1[c] = fmaf(xb[dd], w[c], z1[c]);
                }
            }
        }
        // ---- softmax over the two lanes of a request, contraction with the recall rows, variance
        const int g0 = P.mfirst[a], M = P.mfirst[a + 1] - g0;
#pragma unroll
        for (int t = 0; t < 2; ++t) {
            float(&z)[CT] = t ? z1 : z0;
            float m = z[0];
#pragma unroll
            for (int c = 1; c < CT; ++c) m = fmaxf(m, z[c]);
            m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 16));
            float s = 0.f;
#pragma unroll
            for (int c = 0; c < CT; ++c) { z[c] = expf(z[c] - m); s += z[c]; }
            s += __shfl_xor_sync(0xffffffffu, s, 16);
            const float inv = 1.f / s;
            const bool ok = t ? ok1 : ok0;
            const int64_t req = row0 + s_local[ok ? (t ? p1 : p0) : 0];
            float mean = 0.f, accv[kMaxModelsPerApp];
#pragma unroll
            for (int j = 0; j < kMaxModelsPerApp; ++j) {
                accv[j] = 0.f;
                if (j < M) {
                    float r[CT];
                    load_half_row<CT>(r, smem + L.recall + ((g0 + j) * 2 + h) * CTP);
                    float part = 0.f;
#pragma unroll
                    for (int c = 0; c < CT; ++c) part = fmaf(z[c], r[c], part);
                    part += __shfl_xor_sync(0xffffffffu, part, 16);
                    float aj = part * inv;
                    if (P.prior) {
                        const float ps = P.prior_sum[inst * A + a];
                        aj = (P.prior_dot[(int64_t)inst * P.sumM + g0 + j] + P.kappa * aj) / (ps + P.kappa);
                    }
                    accv[j] = aj;
                    mean += aj;
                }
            }
            mean /= (float)M;
            float var = 0.f;
#pragma unroll
            for (int j = 0; j < kMaxModelsPerApp; ++j)
                if (j < M) var = fmaf(accv[j] - mean, accv[j] - mean, var);
            if (ok && h == 0) {
                float *dst = tb.acc32 + req * P.Mmax;
#pragma unroll
                for (int j = 0; j < kMaxModelsPerApp; ++j)
                    if (j < P.Mmax) dst[j] = accv[j];
                tb.v32[req] = 1.f + var / (float)M;
                if (acc_out) {
                    float *o = acc_out + req * P.Mmax;
#pragma unroll
                    for (int j = 0; j < kMaxModelsPerApp; ++j)
                        if (j < P.Mmax) o[j] = accv[j];
                }
            }
        }
    }
}

}  // namespace sp
