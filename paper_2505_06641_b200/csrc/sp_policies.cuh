// Scheduling policies beyond the application-level greedy rounds of k_sched, all decided on fp64 scores:
//   * k_exact_all      : fp64 scores (Section 4.1, Eq. 9, Eq. 12) and the data-aware label (Section 4.3) of every request,
//                        one warp per request over the whole GPU;
//   * k_sched_groups   : the greedy rounds of Algorithm 1 over data-aware sub-groups ("Enhancements for Grouped
//                        Scheduling": requests of an application with the same predicted label form a group), on one
//                        worker or on several (Section 6: the worker that is free first takes the next batch);
//   * k_exh_*          : the exhaustive branch of Algorithm 1 (number of groups at most the threshold): every order of
//                        the groups times every model choice, one thread per solution;
//   * k_baseline       : the request-level baselines of Section 5.1 (MaxAcc-EDF, LO-EDF, LO-Priority).
// These kernels read acc64 / v64, which k_exact_all fills for all requests first: the decisions are then taken on the
// same numbers (up to the last bits of a sum) as the fp64 definition, and no guard band is needed.
#pragma once

#include "sp_common.cuh"
#include "sp_sched.cuh"

namespace sp {

constexpr int kMaxWorkers = 64;             // workers of the multi-worker rounds
constexpr int kExhMaxGroups = 8;            // groups the exhaustive branch accepts (8! * M^8 solutions at most 2^31)

// ------------------------------------------------------------------------------------------------ fp64 scores of all rows
// One warp per request; zrow scratch in dynamic shared memory: [warps per block][C] doubles.
// gate (optional): the pass runs only when *gate is set (a scheduler asked for it), and skips rows already cached.
__global__ void k_exact_all(DevProfiles P, DevTable tb, int32_t *labels, const int *flags, const int *gate, unsigned long long *stats) {
    extern __shared__ __align__(16) unsigned char dyn[];
    if (flags[1] || (gate && !*gate)) return;
    const int warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    double *zrow = reinterpret_cast<double *>(dyn) + (size_t)warp * P.C;
    unsigned long long done = 0;
    for (int64_t id = (int64_t)blockIdx.x * nwarps + warp; id < tb.n; id += (int64_t)gridDim.x * nwarps) {
        if (gate && tb.exact[id]) continue;
        const int inst = tb.instance ? tb.instance[id] : 0;
        exact_row_core(P, tb, inst, id, zrow, labels ? labels + id : nullptr);
        ++done;
    }
    if (stats && done && (threadIdx.x & 31) == 0) atomicAdd(&stats[3], done);
}

// ------------------------------------------------------------------------------------------------ group queues
// Group of a request: application * GW + label + 1 with GW = C + 1 when sub-groups are on (label -1 = the application's
// unsplit remainder, which therefore comes first), else the application.
struct GroupParams {
    DevProfiles P;
    DevTable tb;
    InstState *state;
    const int32_t *labels;      // [n] or nullptr: groups are the applications
    int64_t *q_id, *q_dl;       // [n] request ids and deadlines in (group, deadline, id) order, instance regions at qstart
    double *q_pw;               // [n] v * exp(-(deadline - Tref)/tau)
    SortKey *keys;              // [n] scratch
    int32_t *g_key, *g_start, *g_head;   // [n + I]: present groups of instance i at [r0 + i, ...): key, first position, head
    int32_t *g_count;           // [I] present groups
    int *flags;
    unsigned long long *stats;
    sp_round_rec *rounds_out;
    int64_t cap;
    int32_t *n_done;
    int sort_cap, bmax, presorted;
    // several workers (Section 6): W > 0 workers with their own latency profiles [W][sumM], clocks and resident models
    // (single-instance contexts); W = 0: the one worker of the profiles
    int W;
    const int64_t *w_alpha, *w_beta, *w_swap;
    int64_t *w_T;
    int32_t *w_L;
};

__device__ __forceinline__ int group_of(const GroupParams &gp, int64_t id) {
    return gp.labels ? gp.tb.app[id] * (gp.P.C + 1) + gp.labels[id] + 1 : gp.tb.app[id];
}

__global__ void k_group_keys(GroupParams gp, int64_t n) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    SortKey k; k.dl = gp.tb.deadline[i]; k.id_rel = (int32_t)i; k.app = group_of(gp, i);
    gp.keys[i] = k;
}

// Sorted queue of one instance and its table of present groups (every thread of the block calls it).  Returns the
// number of groups.  smem_keys: sort_cap SortKey entries of shared memory.
__device__ int build_group_queues(const GroupParams &gp, int inst, SortKey *smem_keys, int64_t tref) {
    __shared__ int s_scan[33];
    __shared__ int s_run;
    const DevTable &tb = gp.tb;
    const int tid = threadIdx.x, NT = blockDim.x, lane = tid & 31, warp = tid >> 5;
    const int64_t r0 = tb.qstart[(int64_t)inst * gp.P.A], r1 = tb.qstart[(int64_t)(inst + 1) * gp.P.A];
    const int n = (int)(r1 - r0);
    SortKey *keys = n <= gp.sort_cap ? smem_keys : gp.keys + r0;
    if (!gp.presorted || n <= gp.sort_cap) {
        for (int t = tid; t < n; t += NT) {
            SortKey k; k.dl = tb.deadline[r0 + t]; k.id_rel = t; k.app = group_of(gp, r0 + t);
            keys[t] = k;
        }
        __syncthreads();
        block_sort(keys, n);
    }
    __syncthreads();
    const int64_t gb = r0 + inst;                         // this instance's slice of the group tables
    if (tid == 0) s_run = 0;
    __syncthreads();
    for (int base = 0; base < n; base += NT) {            // ordered compaction of the positions where a group starts
        const int p = base + tid;
        const bool start = p < n && (p == 0 || keys[p].app != keys[p - 1].app);
        const unsigned bal = __ballot_sync(0xffffffffu, start);
        if (lane == 0) s_scan[warp] = __popc(bal);
        __syncthreads();
        if (warp == 0) {
            int v = lane < (NT >> 5) ? s_scan[lane] : 0, incl = v;
            for (int o = 1; o < 32; o <<= 1) { const int t = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += t; }
            s_scan[lane] = incl - v;
            if (lane == 31) s_scan[32] = incl;
        }
        __syncthreads();
        if (start) {
            const int slot = s_run + s_scan[warp] + __popc(bal & ((1u << lane) - 1u));
            gp.g_key[gb + slot] = keys[p].app; gp.g_start[gb + slot] = p; gp.g_head[gb + slot] = p;
        }
        if (p < n) {
            const int64_t id = r0 + keys[p].id_rel;
            gp.q_id[r0 + p] = id; gp.q_dl[r0 + p] = keys[p].dl;
            gp.q_pw[r0 + p] = prio_weight(tb.v64[id], keys[p].dl, tref, gp.P.tau);
        }
        __syncthreads();
        if (tid == 0) s_run += s_scan[32];
        __syncthreads();
    }
    const int G = s_run;
    if (tid == 0) { gp.g_start[gb + G] = n; gp.g_count[inst] = G; }
    __syncthreads();
    return G;
}

// ------------------------------------------------------------------------------------------------ greedy rounds over sub-groups
struct GroupSchedSmem {
    size_t lat, keys, accs, mem_id, mem_dl, mem_delta, cand_u, cand_e, cand_bp, wbest, end;
    __host__ __device__ GroupSchedSmem(int sort_cap, int Mmax, int bmax, int sumM, int nwarps) {
        size_t o = 0;
        lat = o;    o += (size_t)3 * sumM * sizeof(int64_t);
        keys = o;   o += (size_t)sort_cap * sizeof(SortKey);
        accs = o;   o += (size_t)bmax * Mmax * sizeof(double);
        mem_id = o; o += (size_t)bmax * sizeof(int64_t);
        mem_dl = o; o += (size_t)bmax * sizeof(int64_t);
        mem_delta = o; o += (size_t)bmax * sizeof(int64_t);
        cand_u = o; o += (size_t)kMaxModelsPerApp * kMaxBatchSizes * sizeof(double);
        cand_e = o; o += (size_t)kMaxModelsPerApp * kMaxBatchSizes * sizeof(int64_t);
        wbest = o;  o += (size_t)nwarps * 2 * sizeof(double);
        cand_bp = o; o += (size_t)kMaxModelsPerApp * kMaxBatchSizes * sizeof(int);
        end = (o + 15) & ~(size_t)15;
    }
};

// All rounds of one instance by one thread block, to completion (snapshot mode: every request is pending at the start).
__global__ void __launch_bounds__(1024, 1) k_sched_groups(GroupParams gp) {
    extern __shared__ __align__(16) unsigned char dyn[];
    __shared__ InstState st;
    __shared__ int64_t s_emin[kMaxApps];
    __shared__ int s_retired, s_live, s_best_g, s_best_ci, s_wk;
    __shared__ double s_best_p, s_best_u;
    __shared__ int64_t s_T[kMaxWorkers];
    __shared__ int s_L[kMaxWorkers];
    __shared__ unsigned char s_app_of[kMaxApps * kMaxModelsPerApp];
    const DevProfiles &P = gp.P;
    const DevTable &tb = gp.tb;
    const int inst = blockIdx.x;
    const int W = gp.W;
    const int tid = threadIdx.x, NT = blockDim.x, lane = tid & 31, warp = tid >> 5, nwarps = NT >> 5;
    const int A = P.A, nB = P.nB, Mmax = P.Mmax, bmax = gp.bmax;
    const int GW = gp.labels ? P.C + 1 : 1;
    const GroupSchedSmem L(gp.sort_cap, Mmax, bmax, P.sumM, nwarps);
    int64_t *al = reinterpret_cast<int64_t *>(dyn + L.lat), *be = al + P.sumM, *sw = be + P.sumM;
    double *accs = reinterpret_cast<double *>(dyn + L.accs);
    int64_t *mem_id = reinterpret_cast<int64_t *>(dyn + L.mem_id), *mem_dl = reinterpret_cast<int64_t *>(dyn + L.mem_dl);
    int64_t *mem_delta = reinterpret_cast<int64_t *>(dyn + L.mem_delta);
    double *cand_u = reinterpret_cast<double *>(dyn + L.cand_u);
    int64_t *cand_e = reinterpret_cast<int64_t *>(dyn + L.cand_e);
    int *cand_bp = reinterpret_cast<int *>(dyn + L.cand_bp);
    double *wbest = reinterpret_cast<double *>(dyn + L.wbest);

    if (gp.flags[1]) { if (tid == 0 && gp.n_done) gp.n_done[inst] = 0; return; }
    const int64_t r0 = tb.qstart[(int64_t)inst * A], r1 = tb.qstart[(int64_t)(inst + 1) * A];
    const int n_inst = (int)(r1 - r0);
    const int64_t gb = r0 + inst;
    if (tid == 0) { st = gp.state[inst]; st.Tref = st.T; st.started = 1; s_wk = 0; }
    for (int g = tid; g < P.sumM; g += NT) {
        al[g] = P.lat_alpha[(int64_t)inst * P.sumM + g];
        be[g] = P.lat_beta[(int64_t)inst * P.sumM + g];
        sw[g] = P.swap[(int64_t)inst * P.sumM + g];
        int a2 = 0;
        while (g >= P.mfirst[a2 + 1]) ++a2;
        s_app_of[g] = (unsigned char)a2;
    }
    __syncthreads();
    for (int k = tid; k < W; k += NT) { s_T[k] = st.T; s_L[k] = st.L; }   // every worker starts at the instance's clock
    __syncthreads();
    const int G = build_group_queues(gp, inst, reinterpret_cast<SortKey *>(dyn + L.keys), st.Tref);
    const double tau = P.tau;
    const int64_t reref_ns = tau > 1e8 ? INT64_MAX : (int64_t)(32.0 * tau * 1e9);
    if (tid == 0) s_live = n_inst;
    __syncthreads();
    int rounds_done = 0;
    const int64_t max_iter = 2 * (int64_t)n_inst + 8;
    bool finished = false;
    for (int64_t iter = 0; iter < max_iter; ++iter) {
        if (s_live == 0) { finished = true; break; }
        if (W > 0) {                                     // the worker that is free first takes this round
            if (tid == 0) {
                int wk = 0;
                for (int k = 1; k < W; ++k) if (s_T[k] < s_T[wk]) wk = k;
                s_wk = wk; st.T = s_T[wk]; st.L = s_L[wk];
            }
            __syncthreads();
            for (int g = tid; g < P.sumM; g += NT) {
                al[g] = gp.w_alpha[(int64_t)s_wk * P.sumM + g]; be[g] = gp.w_beta[(int64_t)s_wk * P.sumM + g];
                sw[g] = gp.w_swap[(int64_t)s_wk * P.sumM + g];
            }
            __syncthreads();
        }
        if (st.T - st.Tref > reref_ns) {                 // keep exp((T - Tref)/tau) in range
            for (int p = tid; p < n_inst; p += NT)
                gp.q_pw[r0 + p] = prio_weight(tb.v64[gp.q_id[r0 + p]], gp.q_dl[r0 + p], st.T, tau);
            __syncthreads();
            if (tid == 0) st.Tref = st.T;
            __syncthreads();
        }
        // ---- retire hopeless requests at the head of every group
        if (tid < P.sumM) cand_e[tid] = st.T + (tid != st.L ? sw[tid] : 0) + al[tid] + be[tid] * (int64_t)P.batch[0];
        if (tid == 0) s_retired = 0;
        __syncthreads();
        if (tid < A) {
            int64_t emin = INT64_MAX;
            for (int g = P.mfirst[tid]; g < P.mfirst[tid + 1]; ++g) emin = cand_e[g] < emin ? cand_e[g] : emin;
            s_emin[tid] = emin;
        }
        __syncthreads();
        if (W > 1) {                                     // hopeless = no worker can complete the request in time
            for (int kg = tid; kg < W * P.sumM; kg += NT) {
                const int k = kg / P.sumM, g = kg - k * P.sumM;
                const int64_t e = s_T[k] + (g != s_L[k] ? gp.w_swap[kg] : 0) + gp.w_alpha[kg] + gp.w_beta[kg] * (int64_t)P.batch[0];
                atomicMin(reinterpret_cast<long long *>(&s_emin[s_app_of[g]]), (long long)e);
            }
            __syncthreads();
        }
        for (int s = tid; s < G; s += NT) {
            const int head = gp.g_head[gb + s], tail = gp.g_start[gb + s + 1];
            if (head == tail) continue;
            const int a = gp.g_key[gb + s] / GW, kind = P.pen[a];
            const int64_t emin = s_emin[a];
            int nh = head;
            if (kind == SP_PEN_STEP) {                    // sorted by deadline: the hopeless requests are a prefix
                int lo = head, hi = tail;
                while (lo < hi) { const int mid = (lo + hi) >> 1; if (gp.q_dl[r0 + mid] < emin) lo = mid + 1; else hi = mid; }
                nh = lo;
            } else {
                while (nh < tail) {
                    const int64_t dl = gp.q_dl[r0 + nh];
                    if (!penalty_hopeless(kind, dl, dl - tb.arrival[gp.q_id[r0 + nh]], emin)) break;
                    ++nh;
                }
            }
            for (int p = head; p < nh; ++p) {
                sp_req_rec r; r.status = SP_EXPIRED; r.round = st.round; r.model = -1; r.worker = 0; r.order = 0;
                tb.recs[gp.q_id[r0 + p]] = r;
            }
            if (nh > head) { gp.g_head[gb + s] = nh; atomicAdd(&s_retired, nh - head); }
        }
        __syncthreads();
        if (s_retired > 0) {
            __syncthreads();
            if (tid == 0) { st.exp_since += s_retired; s_live -= s_retired; }
            __syncthreads();
            if (s_live == 0) continue;
        }
        // ---- group priorities (Eq. 14): one warp per group, the best of each warp, then the best of the block
        double bp_ = -INFINITY;
        int bs_ = 0x7fffffff;
        for (int s = warp; s < G; s += nwarps) {
            const int head = gp.g_head[gb + s], tail = gp.g_start[gb + s + 1];
            if (head == tail) continue;
            double part = 0.0;
            for (int p = head + lane; p < tail; p += 32) part += gp.q_pw[r0 + p];
#pragma unroll
            for (int o = 16; o >= 1; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
            const double pr = part / (double)(tail - head);
            if (pr > bp_) { bp_ = pr; bs_ = s; }         // groups are visited in ascending order: ties keep the lowest
        }
        if (lane == 0) { wbest[2 * warp] = bp_; wbest[2 * warp + 1] = (double)bs_; }
        __syncthreads();
        if (tid == 0) {
            double bp2 = -INFINITY; int bs2 = 0x7fffffff;
            for (int w2 = 0; w2 < nwarps; ++w2) {
                const double p2 = wbest[2 * w2]; const int s2 = (int)wbest[2 * w2 + 1];
                if (p2 > bp2 || (p2 == bp2 && s2 < bs2)) { bp2 = p2; bs2 = s2; }
            }
            s_best_g = bs2;
            s_best_p = bp2 * exp((double)(st.T - st.Tref) * 1e-9 / tau);
        }
        __syncthreads();
        // ---- candidates of the chosen group: Eq. 2 summed member by member, in queue order, in fp64
        const int s = s_best_g;
        const int gkey = gp.g_key[gb + s], a = gkey / GW;
        const int head = gp.g_head[gb + s], na = gp.g_start[gb + s + 1] - head, nb = na < bmax ? na : bmax;
        const int m0 = P.mfirst[a], M = P.mfirst[a + 1] - m0, ncand = M * nB, pen = P.pen[a];
        for (int k = tid; k < nb; k += NT) {
            mem_id[k] = gp.q_id[r0 + head + k]; mem_dl[k] = gp.q_dl[r0 + head + k];
            mem_delta[k] = mem_dl[k] - tb.arrival[mem_id[k]];
        }
        __syncthreads();
        for (int k = tid; k < nb * Mmax; k += NT) { const int r = k / Mmax; accs[k] = tb.acc64[mem_id[r] * Mmax + (k - r * Mmax)]; }
        __syncthreads();
        for (int ci = tid; ci < ncand; ci += NT) {
            const int j = ci / nB, bi = ci - j * nB, g = m0 + j;
            const bool valid = bi == 0 || P.batch[bi - 1] < na;
            const int b = P.batch[bi], bp = b < na ? b : na;
            const int64_t e = st.T + (g != st.L ? sw[g] : 0) + al[g] + be[g] * (int64_t)bp;
            double u = 0.0;
            if (valid)
                for (int k = 0; k < bp; ++k) {
                    if (pen == SP_PEN_STEP) { if (!(mem_dl[k] < e)) u = __dadd_rn(u, accs[k * Mmax + j]); }
                    else u = __dadd_rn(u, __dmul_rn(accs[k * Mmax + j], __dsub_rn(1.0, penalty_gamma(pen, mem_dl[k], mem_delta[k], e))));
                }
            cand_u[ci] = valid ? u : -INFINITY; cand_e[ci] = e; cand_bp[ci] = bp;
        }
        __syncthreads();
        if (warp == 0) {
            int best, ncl, mbp; double bu;
            warp_argmax(cand_u, cand_bp, ncand, 0.0, best, bu, ncl, mbp);
            if (lane == 0) { s_best_ci = best; s_best_u = bu; }
        }
        __syncthreads();
        // ---- emit
        const int ci = s_best_ci, bj = ci / nB, bbi = ci - bj * nB, g = m0 + bj, bp = cand_bp[ci];
        const int64_t e = cand_e[ci];
        for (int k = tid; k < bp; k += NT) {
            sp_req_rec r; r.status = SP_SCHEDULED; r.round = st.round; r.model = g; r.worker = s_wk; r.order = st.next_order + k;
            tb.recs[mem_id[k]] = r;
        }
        __syncthreads();
        if (tid == 0) {
            if (gp.rounds_out && rounds_done < gp.cap) {
                sp_round_rec rr;
                rr.instance = inst; rr.round = st.round; rr.app = a; rr.model = g; rr.batch = P.batch[bbi];
                rr.n_members = bp; rr.n_expired = st.exp_since; rr.exact = 3 | (s_wk << 2) | ((gp.labels ? gkey % GW : 0) << 8);
                rr.t_start_ns = st.T; rr.t_end_ns = e; rr.utility = s_best_u; rr.group_priority = s_best_p;
                gp.rounds_out[(int64_t)inst * gp.cap + rounds_done] = rr;
            }
            gp.g_head[gb + s] = head + bp;
            st.T = e; st.L = g; st.round += 1; st.next_order += bp; st.exp_since = 0; s_live -= bp;
            if (W > 0) { s_T[s_wk] = e; s_L[s_wk] = g; }
        }
        ++rounds_done;
        __syncthreads();
    }
    if (tid == 0) {
        if (!finished) dev_error(&gp.flags[0], kDevLimit);
        if (W > 0) {                                     // per-worker clocks; the instance's clock is the last completion
            int64_t tmax = s_T[0];
            for (int k = 0; k < W; ++k) { gp.w_T[k] = s_T[k]; gp.w_L[k] = s_L[k]; tmax = s_T[k] > tmax ? s_T[k] : tmax; }
            st.T = tmax; st.L = s_L[0];
        }
        st.inserted = n_inst;
        for (int a2 = 0; a2 < kMaxApps; ++a2) { st.head[a2] = 0; st.tail[a2] = 0; st.cur[a2] = 0; }
        gp.state[inst] = st;
        if (gp.n_done) gp.n_done[inst] = rounds_done;
        if (rounds_done) atomicAdd(&gp.stats[0], (unsigned long long)rounds_done);
    }
}

// ------------------------------------------------------------------------------------------------ exhaustive branch
struct ExhInfo {                              // written by k_exh_prepare, read by the host and the other two kernels
    int32_t n_groups, status;                 // status: 0 ok, 1 too many groups or solutions
    long long n_solutions, prod_models;
    int32_t models[kExhMaxGroups], first_model[kExhMaxGroups], pen[kExhMaxGroups], app[kExhMaxGroups], label[kExhMaxGroups];
    int32_t start[kExhMaxGroups + 1];
    double best_total;
    long long best_solution;
};

// Single block: the (group, deadline, id) queue of the one instance, its groups, the number of solutions.
__global__ void __launch_bounds__(1024, 1) k_exh_prepare(GroupParams gp, ExhInfo *info) {
    extern __shared__ __align__(16) unsigned char dyn[];
    if (gp.flags[1]) { if (threadIdx.x == 0) { info->status = 1; info->n_groups = 0; info->n_solutions = 0; } return; }
    const int G = build_group_queues(gp, 0, reinterpret_cast<SortKey *>(dyn), gp.state[0].T);
    if (threadIdx.x == 0) {
        const int GW = gp.labels ? gp.P.C + 1 : 1;
        info->n_groups = G; info->status = G > kExhMaxGroups ? 1 : 0;
        double nsol = 1.0; long long prod = 1;
        for (int s = 0; s < G && s < kExhMaxGroups; ++s) {
            const int key = gp.g_key[s], a = key / GW;
            info->models[s] = gp.P.mfirst[a + 1] - gp.P.mfirst[a]; info->first_model[s] = gp.P.mfirst[a];
            info->pen[s] = gp.P.pen[a]; info->app[s] = a; info->label[s] = gp.labels ? key % GW - 1 : -1;
            info->start[s] = gp.g_start[s]; info->start[s + 1] = gp.g_start[s + 1];
            nsol *= (double)info->models[s] * (double)(s + 1); prod *= info->models[s];
        }
        if (nsol > 2147483648.0) info->status = 1;
        info->n_solutions = info->status ? 0 : (long long)nsol; info->prod_models = prod;
        info->best_total = -INFINITY; info->best_solution = -1;
    }
}

// Decodes solution number `sol`: the rank of the group order among the lexicographically sorted permutations is the slow
// part, the model choices (lowest group = slowest digit) the fast part.
__device__ __forceinline__ void exh_decode(const ExhInfo &info, long long sol, int *perm, int *choice) {
    const int G = info.n_groups;
    long long rank = sol / info.prod_models, rest = sol % info.prod_models;
    for (int s = G - 1; s >= 0; --s) { choice[s] = (int)(rest % info.models[s]); rest /= info.models[s]; }
    int avail[kExhMaxGroups];
    for (int s = 0; s < G; ++s) avail[s] = s;
    long long fact = 1;
    for (int s = 2; s < G; ++s) fact *= s;                // (G - 1)!
    for (int pos = 0; pos < G; ++pos) {
        const int k = (int)(rank / fact);
        rank %= fact;
        perm[pos] = avail[k];
        for (int t = k; t + 1 < G - pos; ++t) avail[t] = avail[t + 1];
        if (G - 1 - pos > 0) fact /= (G - 1 - pos);
    }
}

// Total utility (the sum inside Eq. 3) of one solution; every group is served whole in batches of the largest allowed
// size, members in queue order, one running fp64 sum in that order.  emit: also write the schedule.
__device__ double exh_eval(const GroupParams &gp, const ExhInfo &info, const int *perm, const int *choice, bool emit, int *n_rounds) {
    const DevProfiles &P = gp.P;
    const DevTable &tb = gp.tb;
    const int Mmax = P.Mmax, bmax = gp.bmax;
    int64_t T = gp.state[0].T, order = 1;
    int Lm = gp.state[0].L, round = 0;
    double total = 0.0;
    for (int pos = 0; pos < info.n_groups; ++pos) {
        const int s = perm[pos], j = choice[s], m = info.first_model[s] + j, pen = info.pen[s];
        for (int k0 = info.start[s]; k0 < info.start[s + 1]; k0 += bmax) {
            const int bp = min(bmax, info.start[s + 1] - k0);
            const int64_t e = T + (m != Lm ? P.swap[m] : 0) + P.lat_alpha[m] + P.lat_beta[m] * (int64_t)bp;
            double u = 0.0;
            for (int k = 0; k < bp; ++k) {
                const int64_t id = gp.q_id[k0 + k], dl = gp.q_dl[k0 + k];
                const double c = __dmul_rn(tb.acc64[id * Mmax + j], __dsub_rn(1.0, penalty_gamma(pen, dl, dl - tb.arrival[id], e)));
                u = __dadd_rn(u, c);
                total = __dadd_rn(total, c);
                if (emit) {
                    sp_req_rec r; r.status = SP_SCHEDULED; r.round = round; r.model = m; r.worker = 0; r.order = order++;
                    tb.recs[id] = r;
                }
            }
            if (emit && gp.rounds_out && round < gp.cap) {
                sp_round_rec rr;
                rr.instance = 0; rr.round = round; rr.app = info.app[s]; rr.model = m; rr.batch = bmax; rr.n_members = bp;
                rr.n_expired = 0; rr.exact = 3 | ((info.label[s] + 1) << 8); rr.t_start_ns = T; rr.t_end_ns = e;
                rr.utility = u; rr.group_priority = 0.0;
                gp.rounds_out[round] = rr;
            }
            T = e; Lm = m; ++round;
        }
    }
    if (emit) { gp.state[0].T = T; gp.state[0].L = Lm; gp.state[0].round = round; gp.state[0].next_order = order; gp.state[0].started = 1; }
    if (n_rounds) *n_rounds = round;
    return total;
}

// One thread per solution; the best of every block (ties: the lowest solution number) goes to block_best[blockIdx.x].
__global__ void __launch_bounds__(256) k_exh_search(GroupParams gp, const ExhInfo *info_p, double *block_total, long long *block_sol) {
    __shared__ ExhInfo info;
    __shared__ double s_tot[8];
    __shared__ long long s_sol[8];
    if (threadIdx.x == 0) info = *info_p;
    __syncthreads();
    const long long sol = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    double tot = -INFINITY;
    long long mine = 0x7fffffffffffffffLL;
    if (sol < info.n_solutions) {
        int perm[kExhMaxGroups], choice[kExhMaxGroups];
        exh_decode(info, sol, perm, choice);
        tot = exh_eval(gp, info, perm, choice, false, nullptr);
        mine = sol;
    }
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) {
        const double ot = __shfl_xor_sync(0xffffffffu, tot, o);
        const long long os = __shfl_xor_sync(0xffffffffu, mine, o);
        if (ot > tot || (ot == tot && os < mine)) { tot = ot; mine = os; }
    }
    if ((threadIdx.x & 31) == 0) { s_tot[threadIdx.x >> 5] = tot; s_sol[threadIdx.x >> 5] = mine; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < (int)(blockDim.x >> 5); ++w)
            if (s_tot[w] > tot || (s_tot[w] == tot && s_sol[w] < mine)) { tot = s_tot[w]; mine = s_sol[w]; }
        block_total[blockIdx.x] = tot; block_sol[blockIdx.x] = mine;
    }
}

// Single block: best over the blocks, then the schedule of that solution.
__global__ void __launch_bounds__(256) k_exh_finish(GroupParams gp, ExhInfo *info_p, const double *block_total, const long long *block_sol, int n_blocks) {
    __shared__ double s_tot[8];
    __shared__ long long s_sol[8];
    double tot = -INFINITY;
    long long mine = 0x7fffffffffffffffLL;
    for (int b = threadIdx.x; b < n_blocks; b += blockDim.x)
        if (block_total[b] > tot || (block_total[b] == tot && block_sol[b] < mine)) { tot = block_total[b]; mine = block_sol[b]; }
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) {
        const double ot = __shfl_xor_sync(0xffffffffu, tot, o);
        const long long os = __shfl_xor_sync(0xffffffffu, mine, o);
        if (ot > tot || (ot == tot && os < mine)) { tot = ot; mine = os; }
    }
    if ((threadIdx.x & 31) == 0) { s_tot[threadIdx.x >> 5] = tot; s_sol[threadIdx.x >> 5] = mine; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < (int)(blockDim.x >> 5); ++w)
            if (s_tot[w] > tot || (s_tot[w] == tot && s_sol[w] < mine)) { tot = s_tot[w]; mine = s_sol[w]; }
        int n_rounds = 0;
        if (info_p->n_groups > 0 && mine < info_p->n_solutions) {
            int perm[kExhMaxGroups], choice[kExhMaxGroups];
            exh_decode(*info_p, mine, perm, choice);
            tot = exh_eval(gp, *info_p, perm, choice, true, &n_rounds);
        } else tot = 0.0;
        info_p->best_total = tot; info_p->best_solution = mine;
        if (gp.n_done) gp.n_done[0] = n_rounds;
        if (n_rounds) atomicAdd(&gp.stats[0], (unsigned long long)n_rounds);
    }
}

// ------------------------------------------------------------------------------------------------ request-level baselines
struct BaselineParams {
    GroupParams gp;
    int policy;                 // 0 MaxAcc-EDF, 1 LO-EDF, 2 LO-Priority
};

// Order key of a request: the deadline (EDF), or the bit pattern of minus the Eq. 12 priority, which sorts like the
// priority descending (positive doubles order like their bit patterns).
__device__ __forceinline__ int64_t baseline_key(const BaselineParams &bp, int64_t id, int64_t t0) {
    if (bp.policy != 2) return bp.gp.tb.deadline[id];
    return -__double_as_longlong(prio_weight(bp.gp.tb.v64[id], bp.gp.tb.deadline[id], t0, bp.gp.P.tau));
}

__global__ void k_baseline_keys(BaselineParams bp, int64_t n) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    SortKey k; k.dl = baseline_key(bp, i, bp.gp.state[0].T); k.id_rel = (int32_t)i; k.app = 0;
    bp.gp.keys[i] = k;
}

// One block per instance: the block sorts the order keys, then warp 0 walks the requests one by one (lane j scores
// model j of the request's application, warp argmax with ties to the lowest model).
__global__ void __launch_bounds__(1024, 1) k_baseline(BaselineParams bp) {
    extern __shared__ __align__(16) unsigned char dyn[];
    const GroupParams &gp = bp.gp;
    const DevProfiles &P = gp.P;
    const DevTable &tb = gp.tb;
    const int inst = blockIdx.x, tid = threadIdx.x, NT = blockDim.x, lane = tid & 31;
    if (gp.flags[1]) { if (tid == 0 && gp.n_done) gp.n_done[inst] = 0; return; }
    const int64_t r0 = tb.qstart[(int64_t)inst * P.A], r1 = tb.qstart[(int64_t)(inst + 1) * P.A];
    const int n = (int)(r1 - r0);
    SortKey *keys = n <= gp.sort_cap ? reinterpret_cast<SortKey *>(dyn) : gp.keys + r0;
    int64_t T = gp.state[inst].T;
    int Lm = gp.state[inst].L;
    if (!gp.presorted || n <= gp.sort_cap) {
        for (int t = tid; t < n; t += NT) {
            SortKey k; k.dl = baseline_key(bp, r0 + t, T); k.id_rel = t; k.app = 0;
            keys[t] = k;
        }
        __syncthreads();
        block_sort(keys, n);
    }
    __syncthreads();
    if (tid >= 32) return;
    const int Mmax = P.Mmax;
    for (int pos = 0; pos < n; ++pos) {
        const int64_t id = r0 + keys[pos].id_rel;
        const int a = tb.app[id], m0 = P.mfirst[a], M = P.mfirst[a + 1] - m0, pen = P.pen[a];
        const int64_t dl = tb.deadline[id], delta = dl - tb.arrival[id];
        const int g = m0 + (lane < M ? lane : 0);
        const int64_t e = T + (g != Lm ? P.swap[(int64_t)inst * P.sumM + g] : 0) + P.lat_alpha[(int64_t)inst * P.sumM + g]
                          + P.lat_beta[(int64_t)inst * P.sumM + g];
        const double acc = lane < M ? tb.acc64[id * Mmax + lane] : 0.0;
        const double util = __dmul_rn(acc, __dsub_rn(1.0, penalty_gamma(pen, dl, delta, e)));
        const bool feasible = lane < M && !(dl < e);
        const bool any = __ballot_sync(0xffffffffu, feasible) != 0;
        double sc = -INFINITY;
        if (lane < M) sc = bp.policy == 0 ? ((any && !feasible) ? -INFINITY : acc) : util;
        int bj = lane < M ? lane : 0x7fffffff;
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) {
            const double os = __shfl_xor_sync(0xffffffffu, sc, o);
            const int oj = __shfl_xor_sync(0xffffffffu, bj, o);
            if (os > sc || (os == sc && oj < bj)) { sc = os; bj = oj; }
        }
        const int64_t e_best = __shfl_sync(0xffffffffu, (long long)e, bj);
        const double u_best = __shfl_sync(0xffffffffu, util, bj);
        if (lane == 0) {
            sp_req_rec r; r.status = SP_SCHEDULED; r.round = pos; r.model = m0 + bj; r.worker = 0; r.order = pos + 1;
            tb.recs[id] = r;
            if (gp.rounds_out && pos < gp.cap) {
                sp_round_rec rr;
                rr.instance = inst; rr.round = pos; rr.app = a; rr.model = m0 + bj; rr.batch = 1; rr.n_members = 1; rr.n_expired = 0;
                rr.exact = 3; rr.t_start_ns = T; rr.t_end_ns = e_best; rr.utility = u_best;
                rr.group_priority = prio_weight(tb.v64[id], dl, gp.state[inst].T, P.tau);
                gp.rounds_out[(int64_t)inst * gp.cap + pos] = rr;
            }
        }
        T = e_best; Lm = m0 + bj;
    }
    if (lane == 0) {
        InstState *stp = &gp.state[inst];
        stp->T = T; stp->L = Lm; stp->round = n; stp->next_order = (int64_t)n + 1; stp->started = 1; stp->inserted = n;
        if (gp.n_done) gp.n_done[inst] = n;
        if (n) atomicAdd(&gp.stats[0], (unsigned long long)n);
    }
}

}  // namespace sp
