// SneakPeek model of Section 4.1 as the paper builds it: the evidence of a request is the vote of its k nearest labelled
// reference points (training data of the request's application), the posterior is the Dirichlet update of Eq. 10-11
// over those counts, theta its mean; Eq. 9, Eq. 12's variance factor and the Section 4.3 label follow.
//
// Which points are nearest is an integer decision taken on floating-point distances, so the distances are computed the
// way the definition states them: squared Euclidean distance in fp64, summed feature by feature with separate multiplies
// and adds; ties go to the lower reference index.  One warp per request: lane l computes the distances to reference
// points l, l + 32, ... (the reference set is stored feature-major, so the lanes read consecutive addresses), the k
// nearest are then extracted one by one with a warp-wide argmin, and lane j finishes model j.
#pragma once

#include "sp_common.cuh"

namespace sp {

constexpr int kKnnWarps = 4;               // requests per block
constexpr int kKnnMaxK = 1024;

struct KnnParams {
    DevProfiles P;
    DevTable tb;
    int k;
    int64_t R;                  // reference points, grouped by application
    const double *refT;         // [D][R] feature-major, values widened to fp64
    const int32_t *ref_label;   // [R]
    const int64_t *app_start;   // [A + 1] reference points of application a: [app_start[a], app_start[a + 1])
    const double *prior_total;  // [A] sum of the Dirichlet hyper-parameters (nullptr without a prior)
    double *dist;               // [gridDim.x * kKnnWarps][max reference points of an application] scratch
    int64_t dist_stride;
    int32_t *labels;            // [n] out: Section 4.3 label
    float *acc_out;             // optional second destination of the fp32 accuracies
    const int *flags;
};

// Dynamic shared memory: per warp D doubles (the request's features) and C doubles (votes, then theta).
__global__ void __launch_bounds__(kKnnWarps * 32) k_score_knn(KnnParams kp) {
    extern __shared__ __align__(16) unsigned char dyn[];
    if (kp.flags[1]) return;
    const DevProfiles &P = kp.P;
    const DevTable &tb = kp.tb;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int C = P.C, D = P.D, Mmax = P.Mmax;
    double *x = reinterpret_cast<double *>(dyn) + (size_t)warp * (D + C);
    double *theta = x + D;
    double *dist = kp.dist + ((int64_t)blockIdx.x * kKnnWarps + warp) * kp.dist_stride;
    for (int64_t id = (int64_t)blockIdx.x * kKnnWarps + warp; id < tb.n; id += (int64_t)gridDim.x * kKnnWarps) {
        const int a = tb.app[id];
        const int64_t s = kp.app_start[a], Ra = kp.app_start[a + 1] - s;
        for (int d = lane; d < D; d += 32) x[d] = (double)load_feat(tb.feats, P.dtype, id * D + d);
        for (int c = lane; c < C; c += 32) theta[c] = 0.0;
        __syncwarp();
        for (int64_t r0 = 0; r0 < Ra; r0 += 32) {
            const int64_t r = r0 + lane;
            if (r < Ra) {
                double acc = 0.0;
                const double *col = kp.refT + s + r;
                for (int d = 0; d < D; ++d) {
                    const double diff = __dsub_rn(x[d], col[(int64_t)d * kp.R]);
                    acc = __dadd_rn(acc, __dmul_rn(diff, diff));
                }
                dist[r] = acc;
            }
        }
        __syncwarp();
        const int found = (int)(Ra < kp.k ? Ra : kp.k);
        for (int t = 0; t < found; ++t) {                 // the nearest point not taken yet; ties: the lower index
            double bd = INFINITY;
            int64_t bi = INT64_MAX;
            for (int64_t r = lane; r < Ra; r += 32) {
                const double dv = dist[r];
                if (dv < bd) { bd = dv; bi = r; }       // ascending r within a lane: the first of equal distances stays
            }
#pragma unroll
            for (int o = 16; o >= 1; o >>= 1) {
                const double od = __shfl_xor_sync(0xffffffffu, bd, o);
                const int64_t oi = (int64_t)__shfl_xor_sync(0xffffffffu, (long long)bi, o);
                if (od < bd || (od == bd && oi < bi)) { bd = od; bi = oi; }
            }
            if (lane == 0) {
                dist[bi] = INFINITY;                      // (a point at infinite distance is never taken twice: found <= Ra)
                theta[kp.ref_label[s + bi]] += 1.0;
            }
            __syncwarp();
        }
        // posterior mean (Eq. 10-11) over the votes, and the label of Section 4.3
        const double asum = kp.prior_total ? kp.prior_total[a] : 0.0;
        int lab = -1;
        for (int c = lane; c < C; c += 32) {
            double th;
            if (P.prior) th = ((double)P.prior[(int64_t)a * C + c] + theta[c]) / (asum + (double)found);
            else th = found > 0 ? theta[c] / (double)found : 1.0 / (double)C;
            theta[c] = th;
            if (th > 0.5) lab = c;
        }
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) lab = max(lab, __shfl_xor_sync(0xffffffffu, lab, o));
        __syncwarp();
        // Eq. 9: lane j sums model j label by label
        const int m0 = P.mfirst[a], M = P.mfirst[a + 1] - m0;
        double aj = 0.0;
        if (lane < M) {
            const float *rc = P.recall + (int64_t)(m0 + lane) * C;
            for (int c = 0; c < C; ++c) aj = __dadd_rn(aj, __dmul_rn(theta[c], (double)rc[c]));
        }
        double mean = 0.0;
        for (int j = 0; j < M; ++j) mean = __dadd_rn(mean, __shfl_sync(0xffffffffu, aj, j));
        mean = mean / (double)M;
        double var = 0.0;
        for (int j = 0; j < M; ++j) {
            const double dj = __dsub_rn(__shfl_sync(0xffffffffu, aj, j), mean);
            var = __dadd_rn(var, __dmul_rn(dj, dj));
        }
        if (lane < Mmax) {
            const double val = lane < M ? aj : 0.0;
            tb.acc64[id * Mmax + lane] = val;
            tb.acc32[id * Mmax + lane] = (float)val;
            if (kp.acc_out) kp.acc_out[id * Mmax + lane] = (float)val;
        }
        if (lane == 0) {
            const double v = 1.0 + var / (double)M;
            tb.v64[id] = v; tb.v32[id] = (float)v; tb.exact[id] = 1; kp.labels[id] = lab;
        }
        __syncwarp();
    }
}

}  // namespace sp
