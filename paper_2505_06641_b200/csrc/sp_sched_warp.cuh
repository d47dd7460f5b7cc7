// Greedy scheduling rounds with one WARP per instance: the batched mode, where thousands of small independent
// schedulers (a few hundred pending requests each) run in one launch.
//
// It computes exactly what k_sched computes (Section 4.2 and Algorithm 1 of the paper, one batch per round:
// purge, Eq. 14 group priorities, Eq. 2 utilities of every (model variant, batch size) candidate from fp64 prefix
// sums over the deadline-sorted queue head, greedy pick, emit, clock update), but a whole instance lives in one
// warp's slice of shared memory and every step is warp-synchronous: no block barriers, no queue arrays in global
// memory, one global round trip per round (the accuracy rows of the candidate members).  Requests that are
// already hopeless at the starting clock are retired before the sort, so only the survivors are sorted.
// The kernel takes instances that have not started, are not in trace mode and fit the per-warp capacity; it
// leaves the others to k_sched (flags[2] tells that kernel that there is work left for it).
#pragma once

#include "sp_common.cuh"
#include "sp_sched.cuh"

namespace sp {

constexpr int kWarpSchedWarps = 8;          // instances per block

struct WarpSchedSmem {                      // per-warp byte offsets (8-byte aligned pieces)
    size_t dl, pw, ida, pref, end;
    __host__ __device__ WarpSchedSmem(int cap, int Mmax, int bmax) {
        size_t o = 0;
        dl = o;   o += (size_t)cap * sizeof(int64_t);
        pw = o;   o += (size_t)cap * sizeof(double);
        pref = o; o += (size_t)Mmax * (bmax + 1) * sizeof(double);
        ida = o;  o += (size_t)cap * sizeof(uint32_t);          // (application << 24) | request index in the instance
        end = (o + 15) & ~(size_t)15;
    }
};

__device__ __forceinline__ double warp_sum_f64(double v) {
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Ascending (application, deadline, index) order of the packed keys.
__device__ __forceinline__ bool wkey_less(int64_t dl_a, uint32_t ida_a, int64_t dl_b, uint32_t ida_b) {
    const uint32_t app_a = ida_a >> 24, app_b = ida_b >> 24;
    if (app_a != app_b) return app_a < app_b;
    if (dl_a != dl_b) return dl_a < dl_b;
    return ida_a < ida_b;
}

// Bitonic network with ascending comparators only (the first step of every merge mirrors the partner), so a
// length that is not a power of two needs no padding: a partner index >= n stands for +infinity.
__device__ void warp_sort(int64_t *dl, uint32_t *ida, int n) {
    const int lane = threadIdx.x & 31;
    int p2 = 1;
    while (p2 < n) p2 <<= 1;
    for (int k = 2; k <= p2; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
            for (int t = lane; t < (p2 >> 1); t += 32) {
                const int i = ((t & ~(j - 1)) << 1) | (t & (j - 1));
                const int partner = (j == (k >> 1)) ? (i ^ (k - 1)) : (i ^ j);
                if (partner < n && i < n) {
                    const int64_t da = dl[i], db = dl[partner];
                    const uint32_t ia = ida[i], ib = ida[partner];
                    if (wkey_less(db, ib, da, ia)) { dl[i] = db; ida[i] = ib; dl[partner] = da; ida[partner] = ia; }
                }
            }
            __syncwarp();
        }
    }
}

// fp64 re-scoring (exact_row) of the queue positions [k0, k1) of this warp's sorted arrays, where not cached yet.
__device__ void warp_exact_rows(const SchedParams &sp, int inst, int64_t r0, const uint32_t *ida, int k0, int k1,
                                double *zrow, unsigned long long &rows_done) {
    for (int k = k0; k < k1; ++k) {
        const int64_t id = r0 + (ida[k] & 0xFFFFFFu);
        if (!sp.tb.exact[id]) { exact_row(sp, inst, id, zrow); ++rows_done; }
    }
    __syncwarp();
}

__global__ void __launch_bounds__(kWarpSchedWarps * 32)
k_sched_warp(SchedParams sp, int cap) {
    extern __shared__ __align__(16) unsigned char dyn[];
    const DevProfiles &P = sp.P;
    const DevTable &tb = sp.tb;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int inst = blockIdx.x * kWarpSchedWarps + warp;
    if (inst >= P.I || sp.flags[1]) return;
    const int A = P.A, nB = P.nB, Mmax = P.Mmax, bmax = sp.bmax;
    const WarpSchedSmem L(cap, Mmax, bmax);
    unsigned char *mine = dyn + (size_t)warp * L.end;
    int64_t *s_dl = reinterpret_cast<int64_t *>(mine + L.dl);
    double *s_pw = reinterpret_cast<double *>(mine + L.pw);
    uint32_t *s_ida = reinterpret_cast<uint32_t *>(mine + L.ida);
    double *pref = reinterpret_cast<double *>(mine + L.pref);

    const int64_t r0 = tb.gstart[(int64_t)inst * A], r1 = tb.gstart[(int64_t)(inst + 1) * A];
    const int n_inst = (int)(r1 - r0);
    InstState st0 = sp.state[inst];
    if (st0.started || r1 - r0 > cap || r1 - r0 >= (1 << 24)) {      // not this kernel's: leave it to k_sched
        if (lane == 0) sp.flags[2] = 1;
        return;
    }
    int64_t T = st0.T, next_order = st0.next_order;
    const int64_t Tref0 = st0.T;
    int64_t Tref = Tref0;
    int Lm = st0.L, round = st0.round, exp_since = st0.exp_since;
    const double tau = P.tau;
    const int64_t *al = P.lat_alpha + (int64_t)inst * P.sumM;
    const int64_t *be = P.lat_beta + (int64_t)inst * P.sumM;
    const int64_t *sw = P.swap + (int64_t)inst * P.sumM;
    double *zrow = sp.zbuf + (int64_t)inst * sp.zbuf_warps * P.C;

    // earliest completion any candidate of application a can reach from the current clock and resident model
    auto emin_of = [&](int a) -> int64_t {
        int64_t emin = INT64_MAX;
        for (int g = P.mfirst[a]; g < P.mfirst[a + 1]; ++g) {
            const int64_t e = T + (g != Lm ? sw[g] : 0) + al[g] + be[g] * (int64_t)P.batch[0];
            emin = e < emin ? e : emin;
        }
        return emin;
    };

    // ---- requests that are hopeless at the starting clock are retired at once; the others are compacted
    int64_t emin_a = lane < A ? emin_of(lane) : 0;
    int m = 0;                                           // survivors
    for (int k0 = 0; k0 < n_inst; k0 += 32) {
        const int k = k0 + lane;
        bool keep = false;
        int64_t dl = 0;
        int a = 0;
        if (k < n_inst) {
            dl = tb.deadline[r0 + k];
            a = tb.app[r0 + k];
        }
        const int64_t em = __shfl_sync(0xffffffffu, emin_a, a & 31);
        if (k < n_inst) {
            keep = !(dl < em);
            if (!keep) {
                sp_req_rec r; r.status = SP_EXPIRED; r.round = round; r.model = -1; r.pad_ = 0; r.order = 0;
                tb.recs[r0 + k] = r;
            }
        }
        const unsigned mask = __ballot_sync(0xffffffffu, keep);
        if (keep) {
            const int pos = m + __popc(mask & ((1u << lane) - 1u));
            s_dl[pos] = dl;
            s_ida[pos] = ((uint32_t)a << 24) | (uint32_t)k;
        }
        m += __popc(mask);
    }
    exp_since += n_inst - m;
    __syncwarp();
    warp_sort(s_dl, s_ida, m);
    // segment of each application in the sorted array, priority weights relative to the starting clock
    int seg = 0;                                          // lane a <= A: first position whose application is >= a
    if (lane <= A) {
        int lo = 0, hi = m;
        while (lo < hi) { const int mid = (lo + hi) >> 1; if ((int)(s_ida[mid] >> 24) < lane) lo = mid + 1; else hi = mid; }
        seg = lo;
    }
    for (int k = lane; k < m; k += 32)
        s_pw[k] = prio_weight((double)tb.v32[r0 + (s_ida[k] & 0xFFFFFFu)], s_dl[k], Tref, tau);
    __syncwarp();
    int head = seg;                                       // lane a < A: queue of application a is [head, tail)
    const int tail = __shfl_down_sync(0xffffffffu, seg, 1);
    const int seg0 = seg;

    int rounds_done = 0;
    unsigned long long n_exact_u = 0, n_exact_p = 0, n_rows = 0;
    bool finished = false;
    const int max_iter = sp.max_rounds + 2 * n_inst + 8;
    for (int iter = 0; iter < max_iter; ++iter) {
        if (rounds_done >= sp.max_rounds) break;
        int live = lane < A ? tail - head : 0;
        int total = live;
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) total += __shfl_xor_sync(0xffffffffu, total, o);
        if (total == 0) { finished = true; break; }
        // keep exp((T - Tref)/tau) in range: re-reference the stored priority weights now and then
        if ((double)(T - Tref) * 1e-9 / tau > 32.0) {
            for (int a = 0; a < A; ++a) {
                const int h = __shfl_sync(0xffffffffu, head, a), t = __shfl_sync(0xffffffffu, tail, a);
                for (int k = h + lane; k < t; k += 32)
                    s_pw[k] = prio_weight((double)tb.v32[r0 + (s_ida[k] & 0xFFFFFFu)], s_dl[k], T, tau);
            }
            Tref = T;
            __syncwarp();
        }
        // ---------------------------------------------------------------- retire hopeless requests
        int nh = head;
        if (lane < A && tail > head) {
            const int64_t emin = emin_of(lane);
            int lo = head, hi = tail;
            while (lo < hi) { const int mid = (lo + hi) >> 1; if (s_dl[mid] < emin) lo = mid + 1; else hi = mid; }
            nh = lo;
        }
        for (int a = 0; a < A; ++a) {
            const int h = __shfl_sync(0xffffffffu, head, a), h2 = __shfl_sync(0xffffffffu, nh, a);
            for (int k = h + lane; k < h2; k += 32) {
                sp_req_rec r; r.status = SP_EXPIRED; r.round = round; r.model = -1; r.pad_ = 0; r.order = 0;
                tb.recs[r0 + (s_ida[k] & 0xFFFFFFu)] = r;
            }
            exp_since += h2 - h;
        }
        head = nh;
        live = lane < A ? tail - head : 0;
        total = live;
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) total += __shfl_xor_sync(0xffffffffu, total, o);
        if (total == 0) continue;
        // ---------------------------------------------------------------- group priorities (Eq. 14)
        double myP = -INFINITY;                               // lane a: priority of application a
        for (int a = 0; a < A; ++a) {
            const int h = __shfl_sync(0xffffffffu, head, a), t = __shfl_sync(0xffffffffu, tail, a);
            if (t == h) continue;
            double part = 0.0;
            for (int k = h + lane; k < t; k += 32) part += s_pw[k];
            const double S = warp_sum_f64(part);
            if (lane == a) myP = S / (double)(t - h);
        }
        int best_app = -1;
        double best_P = -INFINITY;
        for (int a = 0; a < A; ++a) {
            const double p = __shfl_sync(0xffffffffu, myP, a);
            if (p != -INFINITY && (best_app < 0 || p > best_P)) { best_app = a; best_P = p; }
        }
        const bool contend = lane < A && myP != -INFINITY && myP >= best_P * (1.0 - sp.guard_p);
        const unsigned cmask = __ballot_sync(0xffffffffu, contend);
        double rep_P = best_P * exp((double)(T - Tref) * 1e-9 / tau);
        int round_exact = 0;
        if (__popc(cmask) > 1) {                              // near-tie between groups: decide on fp64 scores
            double exP = -INFINITY;
            for (int a = 0; a < A; ++a) {
                if (!((cmask >> a) & 1u)) continue;
                const int h = __shfl_sync(0xffffffffu, head, a), t = __shfl_sync(0xffffffffu, tail, a);
                warp_exact_rows(sp, inst, r0, s_ida, h, t, zrow, n_rows);
                double part = 0.0;
                for (int k = h + lane; k < t; k += 32) {
                    const double dt = (double)(s_dl[k] - T) * 1e-9 / tau;
                    part += tb.v64[r0 + (s_ida[k] & 0xFFFFFFu)] * exp(-dt);
                }
                const double S = warp_sum_f64(part);
                if (lane == a) exP = S / (double)(t - h);
            }
            best_app = -1;
            for (int a = 0; a < A; ++a) {
                const double p = __shfl_sync(0xffffffffu, exP, a);
                if (((cmask >> a) & 1u) && (best_app < 0 || p > best_P)) { best_app = a; best_P = p; }
            }
            rep_P = best_P;
            round_exact |= 1; ++n_exact_p;
        }
        // ---------------------------------------------------------------- candidates of the chosen group
        const int a = best_app;
        const int qh = __shfl_sync(0xffffffffu, head, a), qt = __shfl_sync(0xffffffffu, tail, a);
        const int na = qt - qh, nb = na < bmax ? na : bmax;
        const int m0 = P.mfirst[a], M = P.mfirst[a + 1] - m0, ncand = M * nB;
        const int64_t *mdl = s_dl + qh;                       // deadlines of the members, ascending
        const uint32_t *mida = s_ida + qh;
        for (int j = lane; j < M; j += 32) pref[(size_t)j * (bmax + 1)] = 0.0;
        {
            double carry[kMaxModelsPerApp];
#pragma unroll
            for (int j = 0; j < kMaxModelsPerApp; ++j) carry[j] = 0.0;
            for (int k0 = 0; k0 < nb; k0 += 32) {             // fp64 prefix sums of the members' accuracies, per model
                const int k = k0 + lane;
                const float *row = tb.acc32 + (r0 + (k < nb ? (int64_t)(mida[k] & 0xFFFFFFu) : 0)) * Mmax;
#pragma unroll
                for (int j = 0; j < kMaxModelsPerApp; ++j) {
                    if (j < M) {
                        double v = k < nb ? (double)row[j] : 0.0;
#pragma unroll
                        for (int o = 1; o < 32; o <<= 1) {
                            const double t = __shfl_up_sync(0xffffffffu, v, o);
                            if (lane >= o) v += t;
                        }
                        v += carry[j];
                        if (k < nb) pref[(size_t)j * (bmax + 1) + k + 1] = v;
                        carry[j] = __shfl_sync(0xffffffffu, v, 31);
                    }
                }
            }
        }
        __syncwarp();
        // best candidate of this lane (lowest index among equals), then of the warp
        double bu = -INFINITY;
        int bi_ = 0x7fffffff;
        for (int ci = lane; ci < ncand; ci += 32) {
            const int j = ci / nB, bi = ci - j * nB, g = m0 + j;
            const int b = P.batch[bi];
            const bool valid = bi == 0 || P.batch[bi - 1] < na;   // a larger size with the same members never wins
            const int bp = b < na ? b : na;
            const int64_t e = T + (g != Lm ? sw[g] : 0) + al[g] + be[g] * (int64_t)bp;
            int lo = 0, hi = bp;                                   // members with deadline < e are late
            while (lo < hi) { const int mid = (lo + hi) >> 1; if (mdl[mid] < e) lo = mid + 1; else hi = mid; }
            const double *pj = pref + (size_t)j * (bmax + 1);
            const double u = valid ? pj[bp] - pj[lo] : -INFINITY;
            if (u > bu) { bu = u; bi_ = ci; }
        }
        double wu = bu;
        int wi = bi_;
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) {
            const double ou = __shfl_xor_sync(0xffffffffu, wu, o);
            const int oi = __shfl_xor_sync(0xffffffffu, wi, o);
            if (ou > wu || (ou == wu && oi < wi)) { wu = ou; wi = oi; }
        }
        // candidates within the guard band of the best one
        const double thr = wu - fabs(wu) * sp.guard_u;
        int ncl = 0, mbp = 0;
        for (int ci = lane; ci < ncand; ci += 32) {
            const int j = ci / nB, bi = ci - j * nB;
            const bool valid = bi == 0 || P.batch[bi - 1] < na;
            const int bp = P.batch[bi] < na ? P.batch[bi] : na;
            if (valid) {
                const int g = m0 + j;
                const int64_t e = T + (g != Lm ? sw[g] : 0) + al[g] + be[g] * (int64_t)bp;
                int lo = 0, hi = bp;
                while (lo < hi) { const int mid = (lo + hi) >> 1; if (mdl[mid] < e) lo = mid + 1; else hi = mid; }
                const double *pj = pref + (size_t)j * (bmax + 1);
                const double u = pj[bp] - pj[lo];
                if (u >= thr) { ++ncl; mbp = max(mbp, bp); }
            }
        }
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) {
            ncl += __shfl_xor_sync(0xffffffffu, ncl, o);
            mbp = max(mbp, __shfl_xor_sync(0xffffffffu, mbp, o));
        }
        if (ncl > 1) {                                        // near-tie between candidates: decide on fp64 scores
            warp_exact_rows(sp, inst, r0, s_ida, qh, qh + mbp, zrow, n_rows);
            bu = -INFINITY; bi_ = 0x7fffffff;
            for (int ci = lane; ci < ncand; ci += 32) {
                const int j = ci / nB, bi = ci - j * nB, g = m0 + j;
                const bool valid = bi == 0 || P.batch[bi - 1] < na;
                const int bp = P.batch[bi] < na ? P.batch[bi] : na;
                if (!valid) continue;
                const int64_t e = T + (g != Lm ? sw[g] : 0) + al[g] + be[g] * (int64_t)bp;
                int lo = 0, hi = bp;
                while (lo < hi) { const int mid = (lo + hi) >> 1; if (mdl[mid] < e) lo = mid + 1; else hi = mid; }
                const double *pj = pref + (size_t)j * (bmax + 1);
                if (!(pj[bp] - pj[lo] >= thr)) continue;
                double u = 0.0;
                for (int k = 0; k < bp; ++k)
                    if (!(mdl[k] < e)) u = __dadd_rn(u, tb.acc64[(r0 + (mida[k] & 0xFFFFFFu)) * Mmax + j]);
                if (u > bu) { bu = u; bi_ = ci; }
            }
            wu = bu; wi = bi_;
#pragma unroll
            for (int o = 16; o >= 1; o >>= 1) {
                const double ou = __shfl_xor_sync(0xffffffffu, wu, o);
                const int oi = __shfl_xor_sync(0xffffffffu, wi, o);
                if (ou > wu || (ou == wu && oi < wi)) { wu = ou; wi = oi; }
            }
            round_exact |= 2; ++n_exact_u;
        }
        // ---------------------------------------------------------------- emit, remove, advance the clock
        const int bj = wi / nB, bbi = wi - bj * nB, g = m0 + bj;
        const int bp = P.batch[bbi] < na ? P.batch[bbi] : na;
        const int64_t e = T + (g != Lm ? sw[g] : 0) + al[g] + be[g] * (int64_t)bp;
        for (int k = lane; k < bp; k += 32) {
            sp_req_rec r; r.status = SP_SCHEDULED; r.round = round; r.model = g; r.pad_ = 0; r.order = next_order + k;
            tb.recs[r0 + (mida[k] & 0xFFFFFFu)] = r;
        }
        if (lane == 0 && sp.rounds_out && rounds_done < sp.cap) {
            sp_round_rec rr;
            rr.instance = inst; rr.round = round; rr.app = a; rr.model = g; rr.batch = P.batch[bbi];
            rr.n_members = bp; rr.n_expired = exp_since; rr.exact = round_exact;
            rr.t_start_ns = T; rr.t_end_ns = e; rr.utility = wu; rr.group_priority = rep_P;
            sp.rounds_out[(int64_t)inst * sp.cap + rounds_done] = rr;
        }
        if (lane == a) head += bp;
        T = e; Lm = g; round += 1; next_order += bp; exp_since = 0;
        ++rounds_done;
        __syncwarp();
    }

    // ---- leave the instance in the state k_sched expects (it resumes from there when rounds are left)
    int live = lane < A ? tail - head : 0;
    int total = live;
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) total += __shfl_xor_sync(0xffffffffu, total, o);
    if (total > 0) {                                          // rounds left for a later call: write the queues out
        for (int a = 0; a < A; ++a) {
            const int h = __shfl_sync(0xffffffffu, head, a), t = __shfl_sync(0xffffffffu, tail, a);
            const int s0 = __shfl_sync(0xffffffffu, seg0, a);
            const int64_t base = tb.gstart[(int64_t)inst * A + a];
            for (int k = h + lane; k < t; k += 32) {
                sp.q_id[0][base + (k - s0)] = r0 + (s_ida[k] & 0xFFFFFFu);
                sp.q_dl[0][base + (k - s0)] = s_dl[k];
                sp.q_pw[0][base + (k - s0)] = s_pw[k];
            }
        }
    }
    InstState *out = &sp.state[inst];
    if (lane < A) { out->head[lane] = head - seg0; out->tail[lane] = tail - seg0; out->cur[lane] = 0; }
    if (lane == 0) {
        if (!finished && rounds_done < sp.max_rounds && total > 0) dev_error(&sp.flags[0], kDevLimit);
        out->T = T; out->next_order = next_order; out->Tref = Tref; out->inserted = n_inst;
        out->L = Lm; out->round = round; out->exp_since = exp_since; out->started = 1;
        if (sp.n_done) sp.n_done[inst] = rounds_done;
        if (rounds_done) atomicAdd(&sp.stats[0], (unsigned long long)rounds_done);
        if (n_exact_u) atomicAdd(&sp.stats[1], n_exact_u);
        if (n_exact_p) atomicAdd(&sp.stats[2], n_exact_p);
        if (n_rows) atomicAdd(&sp.stats[3], n_rows);
    }
}

}  // namespace sp
