// Greedy scheduling rounds with one WARP per instance: the batched mode, where thousands of small independent
// schedulers (a few hundred pending requests each) run in one launch.
//
// It computes what k_sched computes (Section 4.2 and Algorithm 1 of the paper, one batch per round: purge,
// Eq. 14 group priorities, Eq. 2 utilities of every (model variant, batch size) candidate from fp64 prefix sums
// over the deadline-sorted queue head, greedy pick, emit, clock update), but a whole instance lives in one warp's
// slice of shared memory and every step is warp-synchronous: no block barriers, no queue arrays in global memory,
// latency and swap profiles in lane registers, one global round trip per round (the accuracy rows of the
// candidate members).  Requests that are already hopeless at the starting clock are retired before the sort, so
// only the survivors are sorted.
// Applications with a linear or sigmoid penalty (SOFT instantiation) sum Eq. 2 member by member, and their hopeless
// requests leave from the queue head only, as in k_sched.
// A warp takes an instance that has not started, is not in trace mode and fits the per-warp capacity.  The warp
// path does not contain the fp64 re-evaluation of near-ties (which keeps it small): when the two best group
// priorities or candidate utilities of a round are closer than the guard band, the warp writes its queues and
// state out in k_sched's format; after a block barrier the four warps of the block run the block-wide scheduler
// (sched_instance, the body of k_sched) for those instances and for the ones that do not fit a warp.
#pragma once

#include "sp_common.cuh"
#include "sp_sched.cuh"

namespace sp {

constexpr int kWarpSchedWarps = 4;          // instances per block
constexpr int kWarpLoadChunk = 8;           // requests per lane loaded together at the start

struct WarpSchedSmem {                      // per-warp byte offsets (8-byte aligned pieces)
    size_t dl, pw, ida, pref, arr, end;
    __host__ __device__ WarpSchedSmem(int cap, int Mmax, int bmax, bool soft) {
        size_t o = 0;
        dl = o;   o += (size_t)cap * sizeof(int64_t);
        arr = o;  o += soft ? (size_t)cap * sizeof(int64_t) : 0;   // arrival times by request index (soft penalties)
        pw = o;   o += (size_t)cap * sizeof(double);
        // prefix sums (step penalty), or the members' fp32 accuracy rows and relative deadlines (soft penalties)
        const size_t pref_bytes = (size_t)Mmax * (bmax + 1) * sizeof(double);
        const size_t soft_bytes = (((size_t)bmax * Mmax * sizeof(float) + 7) & ~(size_t)7) + (size_t)bmax * sizeof(int64_t);
        pref = o; o += pref_bytes > soft_bytes ? pref_bytes : soft_bytes;
        ida = o;  o += (size_t)cap * sizeof(uint32_t);          // (application << 24) | request index in the instance
        end = (o + 15) & ~(size_t)15;
    }
};

__device__ __forceinline__ double warp_sum_f64(double v) {
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ int warp_sum_i32(int v) {
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ int64_t shfl_i64(int64_t v, int src) {
    return (int64_t)__shfl_sync(0xffffffffu, (long long)v, src);
}

// 1 - gamma of Eq. 2 in fp32 for the warp path's candidate sums.  Both x = (e - d) / delta and 1 - x come from integer
// differences, so the result keeps fp32 relative accuracy also where gamma is close to 1 (no cancellation): far inside
// the guard band under which a round goes to the block-wide scheduler and its fp64 penalty.
__device__ __forceinline__ float penalty_keep_f32(int kind, int64_t d, int64_t delta, int64_t e) {
    if (kind == SP_PEN_STEP || delta <= 0) return d < e ? 0.f : 1.f;
    if (e <= d) return 1.f;
    if (e - d >= delta) return 0.f;
    const float fd = (float)delta;
    const float xm = __fdividef((float)(delta - (e - d)), fd);       // 1 - x
    if (kind == SP_PEN_LINEAR) return xm;
    const float r = __fdividef(xm, __fdividef((float)(e - d), fd));  // (1 - x) / x
    const float r3 = r * r * r;
    // close to x = 1 the fp64 definition 1 - 1 / (1 + r^3) is itself rounded at 1e-16 absolute; there the value is taken
    // from that definition (rare: the request is about to become hopeless), elsewhere r^3 / (1 + r^3) in fp32
    if (r3 < 1e-3f) return (float)__dsub_rn(1.0, penalty_gamma(kind, d, delta, e));
    return r3 < 1e30f ? __fdividef(r3, 1.f + r3) : 1.f;
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
__device__ __forceinline__ void warp_sort(int64_t *dl, uint32_t *ida, int n) {
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

// One instance by one warp.  Returns true when the block-wide scheduler has to take the instance over: a near-tie
// to decide in fp64, more requests than the warp's slice holds, or an instance that had already started.
// MM bounds the models per application and CPL the candidates per lane (models x batch sizes / 32): the loops over
// them are unrolled, and the small instantiation (which also stands for at most 4 applications) keeps the code of a
// round short.
template <int MM, int CPL, bool SOFT>
__device__ bool sched_warp_instance(const SchedParams &sp, const int cap, const int inst, unsigned char *mine) {
    const DevProfiles &P = sp.P;
    const DevTable &tb = sp.tb;
    const int lane = threadIdx.x & 31;
    const int A = P.A, nB = P.nB, Mmax = P.Mmax, bmax = sp.bmax, sumM = P.sumM;
    const WarpSchedSmem L(cap, Mmax, bmax, SOFT);
    int64_t *s_arr = reinterpret_cast<int64_t *>(mine + L.arr);
    int64_t *s_dl = reinterpret_cast<int64_t *>(mine + L.dl);
    double *s_pw = reinterpret_cast<double *>(mine + L.pw);
    uint32_t *s_ida = reinterpret_cast<uint32_t *>(mine + L.ida);
    double *pref = reinterpret_cast<double *>(mine + L.pref);

    const int64_t r0 = tb.qstart[(int64_t)inst * A], r1 = tb.qstart[(int64_t)(inst + 1) * A];
    const int n_inst = (int)(r1 - r0);
    InstState *stp = &sp.state[inst];
    if (stp->started) return true;                                    // not a fresh instance: the block resumes it
    if (r1 - r0 > cap || r1 - r0 >= (1 << 24)) return true;           // does not fit a warp
    int64_t T = stp->T, next_order = stp->next_order;
    int64_t Tref = T;
    int Lm = stp->L, round = stp->round, exp_since = stp->exp_since;
    const double tau = P.tau;
    // lane g: profile of model g; lane a: first model of application a; lane b: allowed batch size b
    const int64_t my_al = lane < sumM ? P.lat_alpha[(int64_t)inst * sumM + lane] : 0;
    const int64_t my_be = lane < sumM ? P.lat_beta[(int64_t)inst * sumM + lane] : 0;
    const int64_t my_sw = lane < sumM ? P.swap[(int64_t)inst * sumM + lane] : 0;
    const int my_mfirst = lane <= A ? P.mfirst[lane] : 0;
    const int my_batch = lane < nB ? P.batch[lane] : 0;
    const int b_min = __shfl_sync(0xffffffffu, my_batch, 0);
    const int my_m0 = my_mfirst, my_M = __shfl_down_sync(0xffffffffu, my_mfirst, 1) - my_mfirst;   // lane a < A
    const int my_pen = (SOFT && lane < A) ? P.pen[lane] : SP_PEN_STEP;                             // lane a < A

    // lane a < A: earliest completion any candidate of application a can reach from the current clock and model
    auto emin_lane = [&]() -> int64_t {
        const int64_t eg = T + (lane != Lm ? my_sw : 0) + my_al + my_be * (int64_t)b_min;      // lane g: model g
        int64_t emin = INT64_MAX;
        for (int j = 0; j < Mmax; ++j) {
            const int64_t e = shfl_i64(eg, (my_m0 + j) & 31);
            if (lane < A && j < my_M) emin = e < emin ? e : emin;
        }
        return emin;
    };

    // ---- requests that are hopeless at the starting clock are retired at once; the others are compacted
    const int64_t emin0 = emin_lane();
    // Soft penalties: hopeless requests leave from the head of the (deadline, index) order only.  The first key of an
    // application that is NOT hopeless bounds that prefix, so one pass over the unsorted requests finds it, and the
    // pass below retires every request ahead of it without sorting them first.
    int64_t first_dl = INT64_MAX;                        // lane a < A: first non-hopeless key of application a
    int first_k = 0x7fffffff;
    if (SOFT) {
        for (int a = 0; a < A; ++a) {
            const int pen_a = __shfl_sync(0xffffffffu, my_pen, a);
            if (pen_a == SP_PEN_STEP) continue;          // uniform
            const int64_t em = shfl_i64(emin0, a);
            int64_t bd = INT64_MAX;
            int bk = 0x7fffffff;
            for (int k = lane; k < n_inst; k += 32) {
                if (tb.app[r0 + k] != a) continue;
                const int64_t dl = tb.deadline[r0 + k];
                if (!penalty_hopeless(pen_a, dl, dl - tb.arrival[r0 + k], em) && (dl < bd || (dl == bd && k < bk))) { bd = dl; bk = k; }
            }
#pragma unroll
            for (int o = 16; o >= 1; o >>= 1) {
                const int64_t od = shfl_i64(bd, lane ^ o);
                const int ok = __shfl_xor_sync(0xffffffffu, bk, o);
                if (od < bd || (od == bd && ok < bk)) { bd = od; bk = ok; }
            }
            if (lane == a) { first_dl = bd; first_k = bk; }
        }
    }
    int m = 0;                                           // survivors
    for (int k0 = 0; k0 < n_inst; k0 += 32 * kWarpLoadChunk) {
        int64_t dlv[kWarpLoadChunk];
        int apv[kWarpLoadChunk];
#pragma unroll
        for (int u = 0; u < kWarpLoadChunk; ++u) {
            const int k = k0 + u * 32 + lane;
            dlv[u] = k < n_inst ? tb.deadline[r0 + k] : 0;
            apv[u] = k < n_inst ? tb.app[r0 + k] : 0;
            if (SOFT && k < n_inst) s_arr[k] = tb.arrival[r0 + k];
        }
#pragma unroll
        for (int u = 0; u < kWarpLoadChunk; ++u) {
            const int k = k0 + u * 32 + lane;
            const int64_t em = shfl_i64(emin0, apv[u] & 31);
            const bool step_app = !SOFT || __shfl_sync(0xffffffffu, my_pen, apv[u] & 31) == SP_PEN_STEP;
            bool gone = step_app && dlv[u] < em;
            if (SOFT) {                                  // ahead of the application's first request that is not hopeless
                const int64_t fd = shfl_i64(first_dl, apv[u] & 31);
                const int fk = __shfl_sync(0xffffffffu, first_k, apv[u] & 31);
                gone = gone || (!step_app && (dlv[u] < fd || (dlv[u] == fd && k < fk)));
            }
            const bool in = k < n_inst, keep = in && !gone;
            if (in && !keep) {
                sp_req_rec r; r.status = SP_EXPIRED; r.round = round; r.model = -1; r.worker = 0; r.order = 0;
                tb.recs[r0 + k] = r;
            }
            const unsigned mask = __ballot_sync(0xffffffffu, keep);
            if (keep) {
                const int pos = m + __popc(mask & ((1u << lane) - 1u));
                s_dl[pos] = dlv[u];
                s_ida[pos] = ((uint32_t)apv[u] << 24) | (uint32_t)k;
            }
            m += __popc(mask);
        }
    }
    exp_since += n_inst - m;
    __syncwarp();
    // sort, then priority weights relative to the starting clock
    float vreg[kWarpLoadChunk * 2];
    const int n_v = (m + 31) >> 5;                        // <= cap / 32
    warp_sort(s_dl, s_ida, m);
    for (int q0 = 0; q0 < n_v; q0 += kWarpLoadChunk * 2) {
#pragma unroll
        for (int u = 0; u < kWarpLoadChunk * 2; ++u) {
            const int k = (q0 + u) * 32 + lane;
            vreg[u] = k < m ? tb.v32[r0 + (s_ida[k] & 0xFFFFFFu)] : 0.f;
        }
#pragma unroll
        for (int u = 0; u < kWarpLoadChunk * 2; ++u) {
            const int k = (q0 + u) * 32 + lane;
            if (k < m) s_pw[k] = (double)vreg[u];
        }
    }
    // the weights in a rolled loop: one copy of the fp64 exponential in the code instead of sixteen
#pragma unroll 1
    for (int k = lane; k < m; k += 32) s_pw[k] = prio_weight(s_pw[k], s_dl[k], Tref, tau);
    int seg = 0;                                          // lane a <= A: first position whose application is >= a
    if (lane <= A) {
        int lo = 0, hi = m;
        while (lo < hi) { const int mid = (lo + hi) >> 1; if ((int)(s_ida[mid] >> 24) < lane) lo = mid + 1; else hi = mid; }
        seg = lo;
    }
    __syncwarp();
    int head = seg;                                       // lane a < A: queue of application a is [head, tail)
    const int tail = __shfl_down_sync(0xffffffffu, seg, 1);
    const int seg0 = seg;

    int rounds_done = 0;
    bool finished = false, handover = false;
    const int max_iter = sp.max_rounds + 2 * n_inst + 8;
    for (int iter = 0; iter < max_iter; ++iter) {
        if (rounds_done >= sp.max_rounds) break;
        if (warp_sum_i32(lane < A ? tail - head : 0) == 0) { finished = true; break; }
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
        const int64_t emin = emin_lane();
        int nh = head;
        if (lane < A && tail > head) {
            if (!SOFT || my_pen == SP_PEN_STEP) {
                int lo = head, hi = tail;
                while (lo < hi) { const int mid = (lo + hi) >> 1; if (s_dl[mid] < emin) lo = mid + 1; else hi = mid; }
                nh = lo;
            } else {                              // soft penalty: the head leaves while it is hopeless
                while (nh < tail) {
                    const int64_t dl = s_dl[nh];
                    if (!penalty_hopeless(my_pen, dl, dl - s_arr[s_ida[nh] & 0xFFFFFFu], emin)) break;
                    ++nh;
                }
            }
        }
        if (warp_sum_i32(lane < A ? nh - head : 0) > 0) {
            for (int a = 0; a < A; ++a) {
                const int h = __shfl_sync(0xffffffffu, head, a), h2 = __shfl_sync(0xffffffffu, nh, a);
                for (int k = h + lane; k < h2; k += 32) {
                    sp_req_rec r; r.status = SP_EXPIRED; r.round = round; r.model = -1; r.worker = 0; r.order = 0;
                    tb.recs[r0 + (s_ida[k] & 0xFFFFFFu)] = r;
                }
                exp_since += h2 - h;
            }
            head = nh;
            if (warp_sum_i32(lane < A ? tail - head : 0) == 0) continue;
        }
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
        if (__popc(__ballot_sync(0xffffffffu, contend)) > 1) { handover = true; break; }   // near-tie between groups
        const double rep_P = best_P * exp((double)(T - Tref) * 1e-9 / tau);
        // ---------------------------------------------------------------- candidates of the chosen group
        const int a = best_app;
        const int qh = __shfl_sync(0xffffffffu, head, a), qt = __shfl_sync(0xffffffffu, tail, a);
        const int na = qt - qh, nb = na < bmax ? na : bmax;
        const int m0 = __shfl_sync(0xffffffffu, my_m0, a), M = __shfl_sync(0xffffffffu, my_M, a), ncand = M * nB;
        const int64_t *mdl = s_dl + qh;                       // deadlines of the members, ascending
        const uint32_t *mida = s_ida + qh;
        const int pen = SOFT ? __shfl_sync(0xffffffffu, my_pen, a) : SP_PEN_STEP;
        float *s_acc = reinterpret_cast<float *>(pref);                                  // soft: [nb][Mmax]
        int64_t *s_delta = reinterpret_cast<int64_t *>(reinterpret_cast<unsigned char *>(pref) +
                                                       (((size_t)bmax * Mmax * sizeof(float) + 7) & ~(size_t)7));
        if (SOFT && pen != SP_PEN_STEP) {          // Eq. 2 member by member: stage the rows and relative deadlines
            for (int k = lane; k < nb; k += 32) {
                const int64_t id = r0 + (int64_t)(mida[k] & 0xFFFFFFu);
                s_delta[k] = mdl[k] - s_arr[mida[k] & 0xFFFFFFu];
                for (int j = 0; j < M; ++j) s_acc[k * Mmax + j] = tb.acc32[id * Mmax + j];
            }
        } else {
        for (int j = lane; j < M; j += 32) pref[(size_t)j * (bmax + 1)] = 0.0;
        {
            double carry[MM];
#pragma unroll
            for (int j = 0; j < MM; ++j) carry[j] = 0.0;
            for (int k0 = 0; k0 < nb; k0 += 32) {             // fp64 prefix sums of the members' accuracies, per model
                const int k = k0 + lane;
                const float *row = tb.acc32 + (r0 + (k < nb ? (int64_t)(mida[k] & 0xFFFFFFu) : 0)) * Mmax;
                float rv[MM];
#pragma unroll
                for (int j = 0; j < MM; ++j) rv[j] = (j < M && k < nb) ? row[j] : 0.f;
#pragma unroll
                for (int j = 0; j < MM; ++j) {
                    if (j < M) {
                        double v = (double)rv[j];
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
        }
        __syncwarp();
        // completion time base and slope of every model, for the candidates: lane g holds model g
        const int64_t base_e = T + (lane != Lm ? my_sw : 0) + my_al;
        double cu[CPL];                          // utilities of this lane's candidates
        double bu = -INFINITY;
        int bi_ = 0x7fffffff;
#pragma unroll
        for (int q = 0; q < CPL; ++q) {
            const int ci = q * 32 + lane;
            cu[q] = -INFINITY;
            if (q * 32 < ncand) {                                  // uniform: shuffles below are warp-wide
                const int cj = ci < ncand ? ci / nB : 0, cb = ci < ncand ? ci - cj * nB : 0, g = m0 + cj;
                const int b = __shfl_sync(0xffffffffu, my_batch, cb);
                const int bprev = __shfl_sync(0xffffffffu, my_batch, cb > 0 ? cb - 1 : 0);
                const int64_t eb = shfl_i64(base_e, g & 31), es = shfl_i64(my_be, g & 31);
                if (ci < ncand) {
                    const bool valid = cb == 0 || bprev < na;      // a larger size with the same members never wins
                    const int bp = b < na ? b : na;
                    const int64_t e = eb + es * (int64_t)bp;
                    double u = -INFINITY;
                    if (SOFT && pen != SP_PEN_STEP) {
                        if (valid) {
                            u = 0.0;
                            for (int k = 0; k < bp; ++k)
                                u += (double)(s_acc[k * Mmax + cj] * penalty_keep_f32(pen, mdl[k], s_delta[k], e));
                        }
                    } else {
                        int lo = 0, hi = bp;                       // members with deadline < e are late
                        while (lo < hi) { const int mid = (lo + hi) >> 1; if (mdl[mid] < e) lo = mid + 1; else hi = mid; }
                        const double *pj = pref + (size_t)cj * (bmax + 1);
                        if (valid) u = pj[bp] - pj[lo];
                    }
                    cu[q] = u;
                    if (u > bu) { bu = u; bi_ = ci; }
                }
            }
        }
        double wu = bu;
        int wi = bi_;
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) {
            const double ou = __shfl_xor_sync(0xffffffffu, wu, o);
            const int oi = __shfl_xor_sync(0xffffffffu, wi, o);
            if (ou > wu || (ou == wu && oi < wi)) { wu = ou; wi = oi; }
        }
        const double thr = wu - fabs(wu) * sp.guard_u;
        int ncl = 0;
#pragma unroll
        for (int q = 0; q < CPL; ++q) ncl += (cu[q] >= thr && cu[q] != -INFINITY) ? 1 : 0;
        if (warp_sum_i32(ncl) > 1) { handover = true; break; }     // near-tie between candidates
        // ---------------------------------------------------------------- emit, remove, advance the clock
        const int bj = wi / nB, bbi = wi - bj * nB, g = m0 + bj;
        const int bsz = __shfl_sync(0xffffffffu, my_batch, bbi);
        const int bp = bsz < na ? bsz : na;
        const int64_t e = shfl_i64(base_e, g & 31) + shfl_i64(my_be, g & 31) * (int64_t)bp;
        for (int k = lane; k < bp; k += 32) {
            sp_req_rec r; r.status = SP_SCHEDULED; r.round = round; r.model = g; r.worker = 0; r.order = next_order + k;
            tb.recs[r0 + (mida[k] & 0xFFFFFFu)] = r;
        }
        if (lane == 0 && sp.rounds_out && rounds_done < sp.cap) {
            sp_round_rec rr;
            rr.instance = inst; rr.round = round; rr.app = a; rr.model = g; rr.batch = bsz;
            rr.n_members = bp; rr.n_expired = exp_since; rr.exact = 0;
            rr.t_start_ns = T; rr.t_end_ns = e; rr.utility = wu; rr.group_priority = rep_P;
            sp.rounds_out[(int64_t)inst * sp.cap + rounds_done] = rr;
        }
        if (lane == a) head += bp;
        T = e; Lm = g; round += 1; next_order += bp; exp_since = 0;
        ++rounds_done;
        __syncwarp();
    }

    // ---- leave the instance in the state k_sched expects: it resumes from there in a later call when rounds
    //      are left, or right after this kernel when a near-tie has to be decided in fp64 (started = 2)
    const int total = warp_sum_i32(lane < A ? tail - head : 0);
    if (total > 0) {
        for (int a = 0; a < A; ++a) {
            const int h = __shfl_sync(0xffffffffu, head, a), t = __shfl_sync(0xffffffffu, tail, a);
            const int s0 = __shfl_sync(0xffffffffu, seg0, a);
            const int64_t base = tb.qstart[(int64_t)inst * A + a];
            for (int k = h + lane; k < t; k += 32) {
                sp.q_id[0][base + (k - s0)] = r0 + (s_ida[k] & 0xFFFFFFu);
                sp.q_dl[0][base + (k - s0)] = s_dl[k];
                sp.q_pw[0][base + (k - s0)] = s_pw[k];
            }
        }
    }
    if (lane < A) { stp->head[lane] = head - seg0; stp->tail[lane] = tail - seg0; stp->cur[lane] = 0; }
    if (lane == 0) {
        if (!finished && !handover && rounds_done < sp.max_rounds && total > 0) dev_error(&sp.flags[0], kDevLimit);
        stp->T = T; stp->next_order = next_order; stp->Tref = Tref; stp->inserted = n_inst;
        stp->L = Lm; stp->round = round; stp->exp_since = exp_since; stp->started = handover ? 2 : 1;
        stp->handed = rounds_done;
        if (sp.n_done) sp.n_done[inst] = rounds_done;
        if (rounds_done) atomicAdd(&sp.stats[0], (unsigned long long)rounds_done);
    }
    return handover;
}

// Four instances per block, one per warp; the instances a warp cannot finish are then run by the whole block with
// the block-wide scheduler (the same code as k_sched), while the other blocks of the grid go on with theirs.
template <int MM, int CPL, bool SOFT>
__global__ void __launch_bounds__(kWarpSchedWarps * 32)
k_sched_warp(SchedParams sp, int cap) {
    extern __shared__ __align__(16) unsigned char dyn[];
    __shared__ int s_takeover[kWarpSchedWarps];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int inst = blockIdx.x * kWarpSchedWarps + warp;
    int take = -1;
    if (inst < sp.P.I) {
        if (sp.flags[1]) {                   // request table failed validation: do nothing
            if (lane == 0 && sp.n_done) sp.n_done[inst] = 0;
        } else {
            const WarpSchedSmem L(cap, sp.P.Mmax, sp.bmax, SOFT);
            if (sched_warp_instance<MM, CPL, SOFT>(sp, cap, inst, dyn + (size_t)warp * L.end)) take = inst;
        }
    }
    if (lane == 0) s_takeover[warp] = take;
    __syncthreads();                         // queues and state of a handed-over instance are in global memory
    for (int w = 0; w < kWarpSchedWarps; ++w) {
        if (s_takeover[w] >= 0) {
            sched_instance<SOFT, (MM <= 8 ? 4 : kMaxApps), false>(sp, s_takeover[w]);
            __syncthreads();
        }
    }
}

}  // namespace sp
