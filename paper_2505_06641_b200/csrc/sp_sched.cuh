// Persistent greedy scheduling kernel: one thread block runs all rounds of one instance on the device.
//
// Per round (Section 4.2 and Algorithm 1 of the paper, one batch per iteration of its loop):
//   1. requests whose arrival time has passed join their application's queue, kept sorted by (deadline, id);
//   2. requests that no candidate of their application could complete in time are retired (utility 0 under
//      the step penalty of Section 5.1);
//   3. group priority (Eq. 14 over Eq. 12) of every non-empty application; the highest goes next;
//   4. every (model variant, batch size) candidate of that application: completion time from the latency
//      profile (+ swap time when the model is not resident), summed member utility (Eq. 2) from fp64 prefix
//      sums over the deadline-sorted head of the queue and a binary search for the members that are late;
//   5. block-wide argmax (ties: lowest model, then smallest batch), emit s_ij, advance clock and queue head.
// Accuracies come from the fp32 scoring kernels.  Whenever the two best group priorities or candidate
// utilities are closer than a guard band (far wider than the fp32 error), the rows involved are re-scored
// in fp64 from the raw features and the decision is taken on those values.
#pragma once

#include "sp_common.cuh"

namespace sp {

struct InstState {
    int64_t T, next_order, Tref, inserted;   // inserted: requests of the instance that have joined a queue
    int32_t L, round, exp_since, started;   // started: 0 fresh, 1 running, 2 handed over by k_sched_warp within this call
    int32_t handed, pad_;                    // rounds of this call done before the hand-over
    int32_t head[kMaxApps], tail[kMaxApps], cur[kMaxApps];   // queue positions relative to the region start
};

struct SortKey { int64_t dl; int32_t id_rel; int32_t app; };  // id_rel: request id - first id of the instance

struct SchedParams {
    DevProfiles P;
    DevTable tb;
    InstState *state;           // [I]
    int64_t *q_id[2];           // [n] request ids, queue regions at gstart[key]
    int64_t *q_dl[2];           // [n] deadlines in queue order
    double *q_pw[2];            // [n] v * exp(-(deadline - Tref)/tau) in queue order
    SortKey *sort_scratch;      // [n]
    double *zbuf;               // [I][warps][C] logits scratch of the fp64 re-evaluation
    int *flags;
    unsigned long long *stats;  // rounds, exact_utility, exact_priority, exact_rows
    int trace_mode;
    double guard_u, guard_p;
    int max_rounds;
    sp_round_rec *rounds_out;
    int64_t cap;
    int32_t *n_done;
    int sort_cap;               // SortKey entries available in shared memory
    int bmax;                   // largest allowed batch size
    int zbuf_warps;             // zbuf rows per instance
    int presorted;              // 1: sort_scratch already holds the sorted keys of the whole (single) instance
    // A near-tie between group priorities re-scores every live request of the contending groups in fp64.  One block
    // does that for a few hundred rows; beyond defer_exact_rows (0 = never) it stops before the round instead, marks the
    // instance (started = 2, handed = rounds done in this call) and raises flags[2]: the host has a grid-wide fp64 pass
    // and a second launch with only_handed = 1 queued behind this kernel, which then finds every row cached.
    int defer_exact_rows;
    int only_handed;            // 1: continue instances that were handed over within this call, leave the others alone
};

__device__ __forceinline__ bool key_less(const SortKey &a, const SortKey &b) {
    if (a.app != b.app) return a.app < b.app;
    if (a.dl != b.dl) return a.dl < b.dl;
    return a.id_rel < b.id_rel;
}

// Sorting network with ascending comparators only (first step of every merge mirrors the partner), so
// a length that is not a power of two needs no padding: a partner index >= n stands for +infinity.
__device__ void block_sort(SortKey *keys, int n) {
    int p2 = 1;
    while (p2 < n) p2 <<= 1;
    for (int k = 2; k <= p2; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
            for (int t = threadIdx.x; t < (p2 >> 1); t += blockDim.x) {
                // t-th pair of this step: low index i has bit j clear
                const int i = ((t & ~(j - 1)) << 1) | (t & (j - 1));
                const int partner = (j == (k >> 1)) ? (i ^ (k - 1)) : (i ^ j);
                if (partner < n && i < n) {
                    const SortKey a = keys[i], b = keys[partner];
                    if (key_less(b, a)) { keys[i] = b; keys[partner] = a; }
                }
            }
            // A step with j <= 32 keeps every pair inside an aligned run of 64 keys, and pairs t .. t + 31 (one
            // warp) cover exactly one such run: between two such steps the warp only has to wait for itself.
            const int next_j = j > 1 ? (j >> 1) : k;              // first step of the next merge has j = k
            if (j <= 32 && next_j <= 32 && (k < p2 || j > 1)) __syncwarp();
            else __syncthreads();
        }
    }
}

// Sort of a short key list by counting: the rank of a key is the number of keys that precede it (keys are
// distinct).  G threads share the comparisons of one key, so every thread of the block works and the longest
// dependent chain is n / G comparisons, where the sorting network above spends log^2 n steps on one or two warps.
// keys and out hold n entries each and do not overlap; the caller synchronises before and after.
__device__ void block_rank_sort(const SortKey *keys, SortKey *out, int n) {
    const int NT = blockDim.x;
    int G = 1;
    while (G < 32 && G * 2 * n <= NT) G <<= 1;
    const int r = threadIdx.x & (G - 1);
    for (int q0 = 0; q0 < n; q0 += NT / G) {          // uniform trip count: the shuffles below need whole warps
        const int q = q0 + threadIdx.x / G;
        int cnt = 0;
        SortKey mine; mine.dl = 0; mine.id_rel = 0; mine.app = 0;
        if (q < n) {
            mine = keys[q];
            for (int m = r; m < n; m += G) cnt += key_less(keys[m], mine) ? 1 : 0;
        }
        for (int o = G >> 1; o >= 1; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
        if (q < n && r == 0) out[cnt] = mine;
    }
}

__device__ __forceinline__ double block_sum(double v, double *red) {
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();
    if (lane == 0) red[wid] = v;
    __syncthreads();
    if (wid == 0) {
        double w = lane < (int)(blockDim.x >> 5) ? red[lane] : 0.0;
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) w += __shfl_xor_sync(0xffffffffu, w, o);
        if (lane == 0) red[32] = w;
    }
    __syncthreads();
    return red[32];
}

// fp64 re-scoring of one request by one warp, written to acc64 / v64.  Plain definition of Section 4.1 /
// Eq. 9 / Eq. 12 with separate multiplies and adds (no fused multiply-add).  zrow: C doubles of scratch owned by the
// warp.  label (optional): receives the request's data-aware sub-group (Section 4.3): the label c whose posterior
// theta_c exceeds one half, or -1 when none does.
__device__ void exact_row_core(const DevProfiles &P, const DevTable &tb, int inst, int64_t id, double *zrow, int32_t *label) {
    const int lane = threadIdx.x & 31;
    const int a = tb.app[id];
    const int64_t head = (int64_t)inst * P.A + a;
    const int C = P.C, D = P.D;
    int64_t frow;
    const void *fmat = feat_matrix(tb, id, frow);
    for (int c0 = 0; c0 < C; c0 += 32) {
        const int c = c0 + lane;
        double z = c < C ? (double)P.bias[head * C + c] : 0.0;
        if (c < C)
            for (int d = 0; d < D; ++d) {
                const double x = (double)load_feat(fmat, P.dtype, frow * D + d);
                const double w = (double)load_feat(P.W, P.dtype, (head * D + d) * C + c);
                z = __dadd_rn(z, __dmul_rn(x, w));
            }
        if (c < C) zrow[c] = z;
    }
    __syncwarp();
    double m = -INFINITY;
    for (int c = lane; c < C; c += 32) m = fmax(m, zrow[c]);
    for (int o = 16; o >= 1; o >>= 1) m = fmax(m, __shfl_xor_sync(0xffffffffu, m, o));
    double s = 0.0;
    for (int c = lane; c < C; c += 32) { const double e = exp(zrow[c] - m); zrow[c] = e; s += e; }
    for (int o = 16; o >= 1; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    __syncwarp();
    double asum = 0.0;
    if (P.prior) {
        double t = 0.0;
        for (int c = lane; c < C; c += 32) t += (double)P.prior[head * C + c];
        for (int o = 16; o >= 1; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
        asum = t;
    }
    int lab = -1;
    for (int c = lane; c < C; c += 32) {
        double th = zrow[c] / s;
        if (P.prior) th = ((double)P.prior[head * C + c] + (double)P.kappa * th) / (asum + (double)P.kappa);
        zrow[c] = th;
        if (th > 0.5) lab = c;
    }
    if (label) {
        for (int o = 16; o >= 1; o >>= 1) lab = max(lab, __shfl_xor_sync(0xffffffffu, lab, o));
        if (lane == 0) *label = lab;
    }
    __syncwarp();
    const int m0 = P.mfirst[a], M = P.mfirst[a + 1] - m0;
    double mean = 0.0, accv[kMaxModelsPerApp];
    for (int j = 0; j < kMaxModelsPerApp; ++j) {
        accv[j] = 0.0;
        if (j < M) {
            const float *r = P.recall + ((int64_t)inst * P.sumM + m0 + j) * C;
            double t = 0.0;
            for (int c = lane; c < C; c += 32) t = __dadd_rn(t, __dmul_rn(zrow[c], (double)r[c]));
            for (int o = 16; o >= 1; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
            accv[j] = t;
            mean += t;
        }
    }
    mean /= (double)M;
    double var = 0.0;
    for (int j = 0; j < kMaxModelsPerApp; ++j)
        if (j < M) var += (accv[j] - mean) * (accv[j] - mean);
    if (lane == 0) {
        for (int j = 0; j < P.Mmax; ++j) tb.acc64[id * P.Mmax + j] = j < M ? accv[j] : 0.0;
        tb.v64[id] = 1.0 + var / (double)M;
        __threadfence_block();
        tb.exact[id] = 1;
    }
    __syncwarp();
}

__device__ __forceinline__ void exact_row(const SchedParams &sp, int inst, int64_t id, double *zrow) {
    exact_row_core(sp.P, sp.tb, inst, id, zrow, nullptr);
}

// Re-scores (if not done before) the requests at queue positions [k0, k1) of one queue buffer.
__device__ void exact_rows(const SchedParams &sp, int inst, const int64_t *qid, int64_t k0, int64_t k1) {
    const int warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    double *zrow = sp.zbuf + ((int64_t)inst * nwarps + warp) * sp.P.C;
    unsigned long long done = 0;
    for (int64_t k = k0 + warp; k < k1; k += nwarps) {
        const int64_t id = qid[k];
        if (!sp.tb.exact[id]) { exact_row(sp, inst, id, zrow); ++done; }
    }
    if ((threadIdx.x & 31) == 0 && done) atomicAdd(&sp.stats[3], done);
    __syncthreads();
}

}  // namespace sp

namespace sp {

// Shared-memory carve-up of k_sched (bytes, 16-byte aligned pieces).
struct SchedSmem {
    size_t lat, part, keys, pref, accs, mem_id, mem_dl, mem_delta, cand_u, cand_e, cand_bp, end;
    __host__ __device__ SchedSmem(int sort_cap, int Mmax, int bmax, int ncand, int sumM, int nwarps) {
        size_t o = 0;
        lat = o;     o += (size_t)3 * sumM * sizeof(int64_t);                 // latency alpha, beta and swap of the instance
        part = o;    o += (size_t)nwarps * kMaxApps * sizeof(double);          // per-warp partial priority sums
        o = (o + 15) & ~(size_t)15;
        keys = o;    o += (size_t)sort_cap * sizeof(SortKey);
        pref = o;    o += (size_t)Mmax * (bmax + 1) * sizeof(double);
        mem_id = o;  o += (size_t)bmax * sizeof(int64_t);
        mem_dl = o;  o += (size_t)bmax * sizeof(int64_t);
        mem_delta = o; o += (size_t)bmax * sizeof(int64_t);
        cand_u = o;  o += (size_t)ncand * sizeof(double);
        cand_e = o;  o += (size_t)ncand * sizeof(int64_t);
        accs = o;    o += (size_t)bmax * Mmax * sizeof(float);
        cand_bp = o; o += (size_t)ncand * sizeof(int);
        end = (o + 15) & ~(size_t)15;
    }
};

// Penalty gamma of Eq. 2 (Section 5.1) for a member with deadline d and relative deadline delta = d - arrival that
// would complete at e.  kind 0: step.  The linear and sigmoid forms are read as x = (e - d) / delta clamped to [0, 1]
// (linear) and 1 / (1 + ((1 - x) / x)^3) in between (sigmoid): the utility degrades from the deadline on and is gone
// once the request is late by its whole relative deadline.  A deadline that is not after the arrival: step.
__device__ __forceinline__ double penalty_gamma(int kind, int64_t d, int64_t delta, int64_t e) {
    if (kind == SP_PEN_STEP || delta <= 0) return d < e ? 1.0 : 0.0;
    if (e <= d) return 0.0;
    if (e - d >= delta) return 1.0;
    const double x = __ddiv_rn((double)(e - d), (double)delta);
    if (kind == SP_PEN_LINEAR) return x;
    const double r = __ddiv_rn(__dsub_rn(1.0, x), x);
    return __ddiv_rn(1.0, __dadd_rn(1.0, __dmul_rn(__dmul_rn(r, r), r)));
}
// No utility is left at completion time e: the request can be retired.  An exact test on the integer times: the
// deadline is missed (step), or e is a whole relative deadline or more after the deadline (soft penalties, x >= 1).
__device__ __forceinline__ bool penalty_hopeless(int kind, int64_t d, int64_t delta, int64_t e) {
    if (kind == SP_PEN_STEP || delta <= 0) return d < e;
    return e - d >= delta;
}

__device__ __forceinline__ double prio_weight(double v, int64_t dl, int64_t tref, double tau) {
    return v * exp(-((double)(dl - tref) * 1e-9 / tau));
}

// Warp 0: argmax of cand_u over [0, ncand) with ties to the lowest index; also counts the entries within
// the relative guard of the maximum and the largest batch among them.  Results are valid in every lane.
__device__ __forceinline__ void warp_argmax(const double *cand_u, const int *cand_bp, int ncand, double guard,
                                            int &best, double &best_u, int &n_close, int &max_bp) {
    const int lane = threadIdx.x & 31;
    double bu = -INFINITY;
    int bi = 0x7fffffff;
    for (int ci = lane; ci < ncand; ci += 32) {
        const double u = cand_u[ci];
        if (u > bu) { bu = u; bi = ci; }
    }
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) {
        const double ou = __shfl_xor_sync(0xffffffffu, bu, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (ou > bu || (ou == bu && oi < bi)) { bu = ou; bi = oi; }
    }
    const double thr = bu - fabs(bu) * guard;
    int cnt = 0, mb = 0;
    for (int ci = lane; ci < ncand; ci += 32) {
        const double u = cand_u[ci];
        if (u >= thr && u != -INFINITY) { ++cnt; mb = max(mb, cand_bp[ci]); }
    }
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) {
        cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
        mb = max(mb, __shfl_xor_sync(0xffffffffu, mb, o));
    }
    best = bi; best_u = bu; n_close = cnt; max_bp = mb;
}

// All rounds of one instance by one thread block (every thread of the block calls it).  SOFT = false leaves the
// linear and sigmoid penalties out of the code (every application has the step penalty): the round loop is a long
// stretch of code that every warp walks through once per round, and what is not there is not fetched.
// MA bounds the applications of the instance: the priority sums are unrolled over it.  LONGQ: the queues are long
// (a large snapshot), so the priority sums keep four loads in flight per thread; short-queue workloads do without
// that code.
template <bool SOFT, int MA, bool LONGQ>
__device__ void sched_instance(const SchedParams &sp, const int inst) {
    extern __shared__ __align__(16) unsigned char dyn[];
    __shared__ InstState st;
    __shared__ double red[33];
    __shared__ double s_P[kMaxApps];
    __shared__ int s_seg[kMaxApps + 2];
    __shared__ int s_lstart[kMaxApps + 1];
    __shared__ int s_lo[kMaxApps], s_hi[kMaxApps], s_pdone[kMaxApps];
    __shared__ int64_t s_emin[kMaxApps];
    __shared__ int64_t s_base[kMaxApps + 1];   // first table row of each application's queue of this instance
    __shared__ unsigned s_ballot[32];
    __shared__ int s_best_app, s_exactP, s_best_ci, s_nclose, s_maxbp;
    __shared__ double s_best_u, s_best_p;
    __shared__ unsigned char s_contend[kMaxApps];

    const DevProfiles &P = sp.P;
    const DevTable &tb = sp.tb;
    const int tid = threadIdx.x, NT = blockDim.x, lane = tid & 31, warp = tid >> 5, nwarps = NT >> 5;
    const int A = P.A, nB = P.nB, Mmax = P.Mmax, bmax = sp.bmax;
    const int ncand_max = kMaxModelsPerApp * kMaxBatchSizes;
    const SchedSmem L(sp.sort_cap, Mmax, bmax, ncand_max, P.sumM, nwarps);
    SortKey *smem_keys = reinterpret_cast<SortKey *>(dyn + L.keys);
    double *pref = reinterpret_cast<double *>(dyn + L.pref);
    float *accs = reinterpret_cast<float *>(dyn + L.accs);
    int64_t *mem_id = reinterpret_cast<int64_t *>(dyn + L.mem_id);
    int64_t *mem_dl = reinterpret_cast<int64_t *>(dyn + L.mem_dl);
    int64_t *mem_delta = reinterpret_cast<int64_t *>(dyn + L.mem_delta);   // relative deadlines (soft penalties only)
    double *cand_u = reinterpret_cast<double *>(dyn + L.cand_u);
    int64_t *cand_e = reinterpret_cast<int64_t *>(dyn + L.cand_e);
    int *cand_bp = reinterpret_cast<int *>(dyn + L.cand_bp);

    if (sp.flags[1]) {                       // request table failed validation: do nothing
        if (tid == 0 && sp.n_done) sp.n_done[inst] = 0;
        return;
    }
    const int64_t r0 = tb.qstart[(int64_t)inst * A], r1 = tb.qstart[(int64_t)(inst + 1) * A];
    const int64_t n_inst = r1 - r0;
    if (tid == 0) st = sp.state[inst];
    if (tid <= A) s_base[tid] = tb.qstart[(int64_t)inst * A + tid];
    __syncthreads();
    if (sp.only_handed) {
        if (st.started != 2) return;            // this call's first launch finished the instance's work
        if (tid == 0) { sp.flags[2] = 0; sp.flags[3] = 1; }   // the grid-wide pass has run: every row of the table is cached
    }

    const double tau = P.tau;
    const int64_t reref_ns = tau > 1e8 ? INT64_MAX : (int64_t)(32.0 * tau * 1e9);   // exp((T - Tref)/tau) stays below e^32
    int64_t *al = reinterpret_cast<int64_t *>(dyn + L.lat), *be = al + P.sumM, *sw = be + P.sumM;
    double *s_part = reinterpret_cast<double *>(dyn + L.part);
    for (int g = tid; g < P.sumM; g += NT) {  // this instance's latency and swap profile, read every round
        al[g] = P.lat_alpha[(int64_t)inst * P.sumM + g];
        be[g] = P.lat_beta[(int64_t)inst * P.sumM + g];
        sw[g] = P.swap[(int64_t)inst * P.sumM + g];
    }
    const int rounds_init = st.started == 2 ? st.handed : 0;   // rounds k_sched_warp ran in this call before handing over
    int rounds_done = rounds_init;
    __syncthreads();
    if (tid == 0 && st.started == 2) st.started = 1;
    __syncthreads();
    unsigned long long n_exact_u = 0, n_exact_p = 0;
    const int64_t max_iter = (int64_t)sp.max_rounds + 2 * n_inst + 8;
    bool finished = false;

    for (int64_t iter = 0; iter < max_iter; ++iter) {
        if (rounds_done >= sp.max_rounds) { finished = true; break; }
        // ---------------------------------------------------------------- 1. arrivals join their queues
        if (tid == 0 && !st.started) { st.started = 1; st.Tref = st.T; }
        __syncthreads();
        int64_t arrived_upto = n_inst;
        if (sp.trace_mode) {
            // Requests are in arrival order: the whole block looks at the next NT arrival times at once (one
            // memory round trip instead of a binary search of dependent loads) and counts those that have passed.
            arrived_upto = st.inserted;
            for (;;) {
                const int64_t k = arrived_upto + tid;
                const int cnt = __syncthreads_count(k < n_inst && tb.arrival[r0 + k] <= st.T);
                arrived_upto += cnt;
                if (cnt < NT) break;
            }
        }
        const int64_t nnew = arrived_upto - st.inserted;
        if (nnew > 0) {
            const int64_t ap = st.inserted;
            const bool presorted = sp.presorted && ap == 0 && nnew == n_inst && nnew > sp.sort_cap;   // sorted by the whole GPU
            SortKey *keys = nnew <= sp.sort_cap ? smem_keys : sp.sort_scratch + r0 + ap;
            if (!presorted) {
                for (int64_t t = tid; t < nnew; t += NT) {
                    const int64_t id = r0 + ap + t;
                    SortKey k; k.dl = tb.deadline[id]; k.id_rel = (int32_t)(ap + t); k.app = tb.app[id];
                    keys[t] = k;
                }
                __syncthreads();
                // short lists: counting sort into the scratch of the candidate step, which is free here
                SortKey *sorted = reinterpret_cast<SortKey *>(dyn + L.pref);
                if (nnew <= sp.sort_cap && nnew * nnew <= 256 * (int64_t)NT && (size_t)nnew * (sizeof(SortKey) + sizeof(int)) <= L.end - L.pref) {
                    block_rank_sort(keys, sorted, (int)nnew);
                    keys = sorted;
                    __syncthreads();
                } else block_sort(keys, (int)nnew);
            }
            if (tid <= A) {                   // first sorted position whose application is >= tid
                int lo = 0, hi = (int)nnew;
                while (lo < hi) { const int mid = (lo + hi) >> 1; if (keys[mid].app < tid) lo = mid + 1; else hi = mid; }
                s_seg[tid] = lo;
            }
            __syncthreads();
            // Merge of every application's new keys into its live queue, all applications at once (one thread per
            // element, so the dependent loads of the binary searches are paid once per call, not once per application).
            if (tid == 0) {                       // live elements of the queues that get new members, flattened
                int tot = 0;
                for (int a = 0; a < A; ++a) {
                    s_lstart[a] = tot;
                    if (s_seg[a + 1] - s_seg[a] > 0) tot += st.tail[a] - st.head[a];
                }
                s_lstart[A] = tot;
            }
            __syncthreads();
            // Few enough new keys: the live elements (which look their place up among the new keys in shared memory)
            // also leave, for every new key, the number of live elements before it; the new keys then need no
            // binary search of dependent loads through the live queue.  The scratch of the candidate step is free here.
            int *live_before = reinterpret_cast<int *>(dyn + L.pref + (size_t)nnew * sizeof(SortKey));
            const bool via_smem = nnew <= sp.sort_cap && (size_t)nnew * (sizeof(SortKey) + sizeof(int)) <= L.end - L.pref;
            for (int f = tid; f < s_lstart[A]; f += NT) {     // live element: count new elements before it
                int a = 0;
                while (f >= s_lstart[a + 1]) ++a;
                const int k = f - s_lstart[a], nn = s_seg[a + 1] - s_seg[a];
                const int64_t base = s_base[a];
                const int head = st.head[a], c = st.cur[a], d = 1 - c;
                const SortKey *nk = keys + s_seg[a];
                const int64_t lidk = sp.q_id[c][base + head + k], dl = sp.q_dl[c][base + head + k], idr = lidk - r0;
                const double pwk = sp.q_pw[c][base + head + k];
                int64_t pdl = 0, pidr = 0;
                if (via_smem && k > 0) { pdl = sp.q_dl[c][base + head + k - 1]; pidr = sp.q_id[c][base + head + k - 1] - r0; }
                int lo = 0, hi = nn;
                while (lo < hi) {
                    const int mid = (lo + hi) >> 1;
                    const bool less = nk[mid].dl < dl || (nk[mid].dl == dl && nk[mid].id_rel < idr);
                    if (less) lo = mid + 1; else hi = mid;
                }
                const int64_t pos = base + head + k + lo;
                sp.q_id[d][pos] = lidk; sp.q_dl[d][pos] = dl; sp.q_pw[d][pos] = pwk;
                if (via_smem) {
                    int plo = 0;                                  // new keys before the previous live element
                    if (k > 0) {
                        hi = lo;
                        while (plo < hi) {
                            const int mid = (plo + hi) >> 1;
                            const bool less = nk[mid].dl < pdl || (nk[mid].dl == pdl && nk[mid].id_rel < pidr);
                            if (less) plo = mid + 1; else hi = mid;
                        }
                    }
                    for (int t = plo; t < lo; ++t) live_before[s_seg[a] + t] = k;
                    if (k == st.tail[a] - head - 1)
                        for (int t = lo; t < nn; ++t) live_before[s_seg[a] + t] = k + 1;
                }
            }
            if (via_smem) __syncthreads();
            for (int t = tid; t < (int)nnew; t += NT) {      // new element: count live elements before it
                const int a = keys[t].app, tl = t - s_seg[a];
                const int64_t base = s_base[a];
                const int head = st.head[a], tail = st.tail[a], nl = tail - head, c = st.cur[a];
                const int64_t dl = keys[t].dl, idr = keys[t].id_rel, id = r0 + idr;
                int lo = 0, buf = c;
                if (nl > 0) {
                    if (via_smem) lo = live_before[t];
                    else {
                        const int64_t *lid = sp.q_id[c] + base + head, *ldl = sp.q_dl[c] + base + head;
                        int hi = nl;
                        while (lo < hi) {
                            const int mid = (lo + hi) >> 1;
                            const int64_t md = ldl[mid];
                            const bool less = md < dl || (md == dl && (lid[mid] - r0) < idr);
                            if (less) lo = mid + 1; else hi = mid;
                        }
                    }
                    buf = 1 - c;
                }
                const int64_t pos = base + (nl > 0 ? head : tail) + tl + lo;
                sp.q_id[buf][pos] = id; sp.q_dl[buf][pos] = dl;
                sp.q_pw[buf][pos] = prio_weight((double)tb.v32[id], dl, st.Tref, tau);
            }
            __syncthreads();
            if (tid == 0) {
                for (int a = 0; a < A; ++a) {
                    const int nn = s_seg[a + 1] - s_seg[a];
                    if (nn == 0) continue;
                    if (st.tail[a] - st.head[a] > 0) st.cur[a] = 1 - st.cur[a];
                    st.tail[a] += nn;
                }
                st.inserted += nnew;
            }
            __syncthreads();
        }
        int64_t live = 0;
        for (int a = 0; a < A; ++a) live += st.tail[a] - st.head[a];
        if (live == 0) {
            if (st.inserted < n_inst) {       // idle: wake at the next arrival
                __syncthreads();
                if (tid == 0) st.T = tb.arrival[r0 + st.inserted];
                __syncthreads();
                continue;
            }
            finished = true;
            break;
        }
        // keep exp((T - Tref)/tau) in range: re-reference the stored priority weights now and then
        if (st.T - st.Tref > reref_ns) {
            for (int a = 0; a < A; ++a) {
                const int64_t base = s_base[a];
                const int c = st.cur[a];
                for (int k = st.head[a] + tid; k < st.tail[a]; k += NT)
                    sp.q_pw[c][base + k] = prio_weight((double)tb.v32[sp.q_id[c][base + k]], sp.q_dl[c][base + k], st.T, tau);
            }
            __syncthreads();
            if (tid == 0) st.Tref = st.T;
            __syncthreads();
        }
        // ---------------------------------------------------------------- 2. retire hopeless requests
        // earliest completion any candidate of the application can reach: every model by its own thread, then the
        // minimum per application (the candidate table is free at this point of the round)
        if (tid < P.sumM) cand_e[tid] = st.T + (tid != st.L ? sw[tid] : 0) + al[tid] + be[tid] * (int64_t)P.batch[0];
        __syncthreads();
        if (tid < A) {
            const int a = tid;
            int64_t emin = INT64_MAX;
            for (int g = P.mfirst[a]; g < P.mfirst[a + 1]; ++g) emin = cand_e[g] < emin ? cand_e[g] : emin;
            s_emin[a] = emin;
            s_lo[a] = st.head[a]; s_hi[a] = st.tail[a]; s_pdone[a] = st.tail[a] == st.head[a];
        }
        __syncthreads();
        // The hopeless requests at the head of every queue are retired.  Each application gets per = NT / A threads
        // that look at per queue positions at once (one memory round trip per pass):
        //   - window: the next per positions behind lo; the leading hopeless ones are counted.  Soft penalties only
        //     ever use windows (hopeless depends on the relative deadline too, so it is not a sorted prefix) and slide
        //     the window while it is hopeless throughout.
        //   - samples (step penalty, after a first window that was hopeless throughout, more than per positions left):
        //     the queue is sorted by deadline, so the hopeless requests are a prefix; per evenly spaced samples narrow
        //     [lo, hi) by a factor per + 1 per pass.
        for (int pass = 0; pass < max_iter; ++pass) {
            const int per = NT / A, a = tid / per, j = tid - a * per;
            bool late = false;
            if (a < A && !s_pdone[a]) {
                const int lo = s_lo[a], hi = s_hi[a], span = hi - lo, kind = SOFT ? P.pen[a] : SP_PEN_STEP;
                const bool window = pass == 0 || kind != SP_PEN_STEP || span <= per;
                const int k = window ? lo + j : lo + (int)(((int64_t)(j + 1) * span) / (per + 1));
                if (k < hi) {
                    const int64_t gb = s_base[a];
                    const int64_t dl = sp.q_dl[st.cur[a]][gb + k];
                    const int64_t delta = kind == SP_PEN_STEP ? 0 : dl - tb.arrival[sp.q_id[st.cur[a]][gb + k]];
                    late = penalty_hopeless(kind, dl, delta, s_emin[a]);
                }
            }
            const unsigned bal = __ballot_sync(0xffffffffu, late);
            if (lane == 0) s_ballot[warp] = bal;
            __syncthreads();
            if (tid < A && !s_pdone[tid]) {
                const int a2 = tid, lo = s_lo[a2], hi = s_hi[a2], span = hi - lo, kind = SOFT ? P.pen[a2] : SP_PEN_STEP;
                const bool window = pass == 0 || kind != SP_PEN_STEP || span <= per;
                int cnt = 0;                      // leading hopeless positions among the per looked at
                for (int t2 = a2 * per, end = t2 + per; t2 < end;) {
                    const unsigned clear = ~(s_ballot[t2 >> 5] >> (t2 & 31));
                    const int avail = min(32 - (t2 & 31), end - t2), run = clear ? __ffs(clear) - 1 : 32;
                    if (run < avail) { cnt += run; break; }
                    cnt += avail; t2 += avail;
                }
                if (window) {
                    if (cnt == per && lo + per < hi) s_lo[a2] = lo + per;          // hopeless throughout: slide on
                    else { s_lo[a2] = lo + cnt; s_pdone[a2] = 1; }
                } else {                          // sample j2 sits at lo + (j2 + 1) span / (per + 1)
                    const int below = cnt == 0 ? lo : lo + (int)(((int64_t)cnt * span) / (per + 1)) + 1;
                    const int above = cnt == per ? hi : lo + (int)(((int64_t)(cnt + 1) * span) / (per + 1));
                    s_lo[a2] = below; s_hi[a2] = above;
                    if (below >= above) s_pdone[a2] = 1;
                }
            }
            __syncthreads();
            bool all_done = true;
            for (int a2 = 0; a2 < A; ++a2) all_done = all_done && s_pdone[a2];
            if (all_done) break;
            __syncthreads();
        }
        int n_retired = 0;                    // s_lo is the new head of every queue
        for (int a2 = 0; a2 < A; ++a2) n_retired += s_lo[a2] - st.head[a2];
        if (n_retired > 0) {
            for (int a2 = 0; a2 < A; ++a2) {
                const int64_t *qid = sp.q_id[st.cur[a2]] + s_base[a2];
                for (int k = st.head[a2] + tid; k < s_lo[a2]; k += NT) {
                    sp_req_rec r; r.status = SP_EXPIRED; r.round = st.round; r.model = -1; r.worker = 0; r.order = 0;
                    tb.recs[qid[k]] = r;
                }
            }
            __syncthreads();
            if (tid == 0) {
                for (int a2 = 0; a2 < A; ++a2) st.head[a2] = s_lo[a2];
                st.exp_since += n_retired;
            }
            __syncthreads();
        }
        live = 0;
        for (int a = 0; a < A; ++a) live += st.tail[a] - st.head[a];
        if (live == 0) continue;
        // ---------------------------------------------------------------- 3. group priorities (Eq. 14)
        {
            // partial sums of every application first (their loads are in flight together), then one reduction
            double part[MA];
#pragma unroll
            for (int a = 0; a < MA; ++a) {
                part[a] = 0.0;
                if (a < A) {
                    const double *pw = sp.q_pw[st.cur[a]] + s_base[a];
                    int k = st.head[a] + tid;
                    if (LONGQ) {                      // read at the SM's bandwidth, not at one round trip per element
                        const int tail = st.tail[a];
                        double p1 = 0.0, p2 = 0.0, p3 = 0.0;
                        for (; k + 3 * NT < tail; k += 4 * NT) {
                            part[a] += pw[k]; p1 += pw[k + NT]; p2 += pw[k + 2 * NT]; p3 += pw[k + 3 * NT];
                        }
                        part[a] += (p1 + p2) + p3;
                    }
                    for (; k < st.tail[a]; k += NT) part[a] += pw[k];
                }
            }
#pragma unroll
            for (int a = 0; a < MA; ++a) {
                if (a < A) {
                    double v = part[a];
#pragma unroll
                    for (int o = 16; o >= 1; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
                    if (lane == 0) s_part[warp * kMaxApps + a] = v;
                }
            }
            __syncthreads();
            if (tid < A) {
                const int na = st.tail[tid] - st.head[tid];
                double S = 0.0;
                for (int w2 = 0; w2 < nwarps; ++w2) S += s_part[w2 * kMaxApps + tid];
                s_P[tid] = na > 0 ? S / (double)na : -INFINITY;
            }
        }
        __syncthreads();
        if (tid == 0) {
            int ba = -1;
            for (int a = 0; a < A; ++a)
                if (s_P[a] != -INFINITY && (ba < 0 || s_P[a] > s_P[ba])) ba = a;
            int close = 0;
            for (int a = 0; a < A; ++a) {
                const bool c = s_P[a] != -INFINITY && s_P[a] >= s_P[ba] * (1.0 - sp.guard_p);
                s_contend[a] = c; close += c;
            }
            s_best_app = ba;
            s_exactP = close > 1;
            s_best_p = s_P[ba] * exp((double)(st.T - st.Tref) * 1e-9 / tau);
        }
        __syncthreads();
        int round_exact = 0;
        if (s_exactP && sp.defer_exact_rows > 0 && !sp.flags[3]) {
            int64_t rows = 0;
            for (int a = 0; a < A; ++a) rows += s_contend[a] ? st.tail[a] - st.head[a] : 0;
            if (rows > sp.defer_exact_rows) {   // too many rows for one block: leave them to the whole GPU and resume
                __syncthreads();
                if (tid == 0) { st.started = 2; st.handed = rounds_done; sp.flags[2] = 1; }
                __syncthreads();
                finished = true;
                break;
            }
        }
        if (s_exactP) {                        // near-tie between groups: decide on fp64 scores
            for (int a = 0; a < A; ++a) {
                if (!s_contend[a]) continue;
                const int64_t base = s_base[a];
                const int c = st.cur[a];
                exact_rows(sp, inst, sp.q_id[c] + base, st.head[a], st.tail[a]);
                double part = 0.0;
                for (int k = st.head[a] + tid; k < st.tail[a]; k += NT) {
                    const double dt = (double)(sp.q_dl[c][base + k] - st.T) * 1e-9 / tau;
                    part += tb.v64[sp.q_id[c][base + k]] * exp(-dt);
                }
                const double S = block_sum(part, red);
                if (tid == 0) s_P[a] = S / (double)(st.tail[a] - st.head[a]);
            }
            __syncthreads();
            if (tid == 0) {
                int ba = -1;
                for (int a = 0; a < A; ++a)
                    if (s_contend[a] && (ba < 0 || s_P[a] > s_P[ba])) ba = a;
                s_best_app = ba; s_best_p = s_P[ba];
            }
            __syncthreads();
            round_exact |= 1; ++n_exact_p;
        }
        // ---------------------------------------------------------------- 4. candidates of the chosen group
        const int a = s_best_app;
        const int64_t base = s_base[a];
        const int c = st.cur[a], head = st.head[a], na = st.tail[a] - head;
        const int nb = na < bmax ? na : bmax;
        const int m0 = P.mfirst[a], M = P.mfirst[a + 1] - m0, ncand = M * nB;
        for (int k = tid; k < nb; k += NT) {
            mem_id[k] = sp.q_id[c][base + head + k];
            mem_dl[k] = sp.q_dl[c][base + head + k];
            if (SOFT && P.pen[a] != SP_PEN_STEP) mem_delta[k] = mem_dl[k] - tb.arrival[mem_id[k]];
        }
        const int pen = SOFT ? P.pen[a] : SP_PEN_STEP;
        __syncthreads();
        for (int k = tid; k < nb * Mmax; k += NT) {
            const int r = k / Mmax, j = k - r * Mmax;
            accs[k] = tb.acc32[mem_id[r] * Mmax + j];
        }
        __syncthreads();
        for (int j = warp; j < M; j += nwarps) {      // fp64 prefix sums of the members' accuracies, per model
            double *pj = pref + (size_t)j * (bmax + 1);
            double carry = 0.0;
            if (lane == 0) pj[0] = 0.0;
            for (int k0 = 0; k0 < nb; k0 += 32) {
                const int k = k0 + lane;
                double v = k < nb ? (double)accs[k * Mmax + j] : 0.0;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const double t = __shfl_up_sync(0xffffffffu, v, o);
                    if (lane >= o) v += t;
                }
                v += carry;
                if (k < nb) pj[k + 1] = v;
                carry = __shfl_sync(0xffffffffu, v, 31);
            }
        }
        __syncthreads();
        for (int ci = tid; ci < ncand; ci += NT) {
            const int j = ci / nB, bi = ci - j * nB, g = m0 + j;
            const int b = P.batch[bi];
            const bool valid = bi == 0 || P.batch[bi - 1] < na;   // a larger size with the same members never wins
            const int bp = b < na ? b : na;
            const int64_t e = st.T + (g != st.L ? sw[g] : 0) + al[g] + be[g] * (int64_t)bp;
            double u;
            if (pen == SP_PEN_STEP) {
                int lo = 0, hi = bp;                               // members with deadline < e are late
                while (lo < hi) { const int mid = (lo + hi) >> 1; if (mem_dl[mid] < e) lo = mid + 1; else hi = mid; }
                const double *pj = pref + (size_t)j * (bmax + 1);
                u = pj[bp] - pj[lo];
            } else {                                               // Eq. 2 member by member: acc * (1 - gamma)
                u = 0.0;
                if (valid)
                    for (int k = 0; k < bp; ++k)
                        u = __dadd_rn(u, __dmul_rn((double)accs[k * Mmax + j], __dsub_rn(1.0, penalty_gamma(pen, mem_dl[k], mem_delta[k], e))));
            }
            cand_u[ci] = valid ? u : -INFINITY;
            cand_e[ci] = e; cand_bp[ci] = bp;
        }
        __syncthreads();
        if (warp == 0) {
            int best, ncl, mbp; double bu;
            warp_argmax(cand_u, cand_bp, ncand, sp.guard_u, best, bu, ncl, mbp);
            if (lane == 0) { s_best_ci = best; s_best_u = bu; s_nclose = ncl; s_maxbp = mbp; }
        }
        __syncthreads();
        if (s_nclose > 1) {                    // near-tie between candidates: decide on fp64 scores
            const double thr = s_best_u - fabs(s_best_u) * sp.guard_u;
            exact_rows(sp, inst, sp.q_id[c] + base, head, head + s_maxbp);
            for (int ci = tid; ci < ncand; ci += NT) {
                const double u32 = cand_u[ci];
                double u = -INFINITY;
                if (u32 >= thr && u32 != -INFINITY) {
                    const int j = ci / nB, bp = cand_bp[ci];
                    const int64_t e = cand_e[ci];
                    u = 0.0;
                    for (int k = 0; k < bp; ++k) {
                        if (pen == SP_PEN_STEP) { if (!(mem_dl[k] < e)) u = __dadd_rn(u, tb.acc64[mem_id[k] * Mmax + j]); }
                        else u = __dadd_rn(u, __dmul_rn(tb.acc64[mem_id[k] * Mmax + j], __dsub_rn(1.0, penalty_gamma(pen, mem_dl[k], mem_delta[k], e))));
                    }
                }
                cand_u[ci] = u;
            }
            __syncthreads();
            if (warp == 0) {
                int best, ncl, mbp; double bu;
                warp_argmax(cand_u, cand_bp, ncand, 0.0, best, bu, ncl, mbp);
                if (lane == 0) { s_best_ci = best; s_best_u = bu; }
            }
            __syncthreads();
            round_exact |= 2; ++n_exact_u;
        }
        // ---------------------------------------------------------------- 5. emit, remove, advance the clock
        const int ci = s_best_ci, bj = ci / nB, bbi = ci - bj * nB, g = m0 + bj;
        const int bp = cand_bp[ci];
        const int64_t e = cand_e[ci];
        for (int k = tid; k < bp; k += NT) {
            sp_req_rec r; r.status = SP_SCHEDULED; r.round = st.round; r.model = g; r.worker = 0;
            r.order = st.next_order + k;
            tb.recs[mem_id[k]] = r;
        }
        __syncthreads();
        if (tid == 0) {
            if (sp.rounds_out && rounds_done < sp.cap) {
                sp_round_rec rr;
                rr.instance = inst; rr.round = st.round; rr.app = a; rr.model = g; rr.batch = P.batch[bbi];
                rr.n_members = bp; rr.n_expired = st.exp_since; rr.exact = round_exact;
                rr.t_start_ns = st.T; rr.t_end_ns = e; rr.utility = s_best_u; rr.group_priority = s_best_p;
                sp.rounds_out[(int64_t)inst * sp.cap + rounds_done] = rr;
            }
            st.head[a] += bp; st.T = e; st.L = g; st.round += 1; st.next_order += bp; st.exp_since = 0;
        }
        ++rounds_done;
        __syncthreads();
    }
    if (tid == 0) {
        if (!finished && rounds_done < sp.max_rounds) dev_error(&sp.flags[0], kDevLimit);
        sp.state[inst] = st;
        if (sp.n_done) sp.n_done[inst] = rounds_done;
        if (rounds_done > rounds_init) atomicAdd(&sp.stats[0], (unsigned long long)(rounds_done - rounds_init));
        if (n_exact_u) atomicAdd(&sp.stats[1], n_exact_u);
        if (n_exact_p) atomicAdd(&sp.stats[2], n_exact_p);
    }
}

template <bool SOFT, int MA, bool LONGQ>
__global__ void __launch_bounds__(1024, 1) k_sched(SchedParams sp) { sched_instance<SOFT, MA, LONGQ>(sp, blockIdx.x); }

}  // namespace sp
