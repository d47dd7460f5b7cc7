/*
 * SneakPeek scoring-and-selection ORACLE  --  TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, fp64 CPU statement of what the scheduler's per-round hot path computes,
 * written from the paper (arXiv 2505.06641).  It exists so that the CUDA library can be
 * checked against something that was not derived from it: only tests, the smoke check and
 * the benchmark's CPU-baseline leg may call it.  It shares no code, header, table or helper
 * with the CUDA path.  Nothing here is blocked, fused or reordered beyond what the cited
 * passage states; time is int64 nanoseconds so every deadline test and clock update is exact.
 * Build: gcc -O2 -ffp-contract=off -fopenmp -shared -fPIC.
 *
 * Parity pins (tests/test_oracle_pins.py): Dirichlet worked example of Section 4.1, the
 * Eq. 7 == Eq. 9 identity, one-hot / uniform special cases, scipy softmax, the population
 * variance footnote of Eq. 12, an independent replay of Eq. 1-3 over the emitted schedule,
 * literal Algorithm 1 on one-batch groups, brute force over all pick sequences on tiny queues.
 * Parity UNPINNED by the paper (readings of points it leaves open, pinned only by their
 * stated definition): the purge rule for hopeless requests, deadline order inside a group,
 * batch-size candidates with l(m,b) = alpha + beta*b and a separate swap cost, and the linear
 * and sigmoid penalties (Section 5.1 prints them garbled; orc_penalty() states the reading and
 * is pinned only at gamma(e = d) = 0, gamma(half way) = 1/2, gamma(>= relative deadline late) = 1
 * and monotonicity).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORC_F32 = 0, ORC_BF16 = 1 };
enum { ORC_PENDING = 0, ORC_SCHEDULED = 1, ORC_EXPIRED = 2 };
enum { ORC_PEN_STEP = 0, ORC_PEN_LINEAR = 1, ORC_PEN_SIGMOID = 2 };

typedef struct {
    int32_t n_instances, n_apps, n_classes, feat_dim, feat_dtype;
    const int32_t *models_per_app;   /* [A] */
    const void *head_w;              /* [I][A][D][C], C fastest; float or bf16 bits */
    const float *head_b;             /* [I][A][C] */
    const float *prior_alpha;        /* [I][A][C] or NULL */
    double evidence_k;               /* kappa: weight of the soft evidence y = kappa * p */
    const float *recall;             /* [I][sumM][C] */
    const int64_t *lat_alpha_ns, *lat_beta_ns, *swap_ns; /* [I][sumM] */
    const int32_t *batch_sizes;      /* [nB] ascending */
    int32_t n_batch_sizes;
    double prio_time_scale_s;        /* tau of exp(-(d - T)/tau) */
    const int32_t *penalty_kind;     /* [A] ORC_PEN_*, or NULL = step for every application */
} orc_profiles;

typedef struct {
    int32_t instance, round, app, model, batch, n_members, n_expired, pad_;
    int64_t t_start_ns, t_end_ns;
    double utility, group_priority;
    double util_margin;   /* (U1-U2)/U1 over candidates of the chosen group with a different value; +inf if none */
    double prio_margin;   /* (P1-P2)/P1 over the other non-empty groups; +inf if none */
} orc_round_rec;

typedef struct {
    int32_t status, round, model, pad_;
    int64_t order;
} orc_req_rec;

static double widen(const void *base, int dtype, int64_t idx)
{
    if (dtype == ORC_BF16) {
        uint32_t bits = ((uint32_t)((const uint16_t *)base)[idx]) << 16;
        float f;
        memcpy(&f, &bits, sizeof f);
        return (double)f;
    }
    return (double)((const float *)base)[idx];
}

static int sum_models(const orc_profiles *p)
{
    int s = 0;
    for (int a = 0; a < p->n_apps; ++a) s += p->models_per_app[a];
    return s;
}

static int max_models(const orc_profiles *p)
{
    int s = 0;
    for (int a = 0; a < p->n_apps; ++a) if (p->models_per_app[a] > s) s = p->models_per_app[a];
    return s;
}

static int first_model(const orc_profiles *p, int app)
{
    int s = 0;
    for (int a = 0; a < app; ++a) s += p->models_per_app[a];
    return s;
}

/* ---------------------------------------------------------------------------------------------
 * Scoring of one request.
 *   logits + softmax : the SneakPeek model of Definition 4.1.1, here a linear head whose
 *                      softmax output p is the (soft) evidence.
 *   theta            : mean of the Dirichlet posterior of Eq. 10-11 with evidence y = kappa*p:
 *                      theta_c = (alpha_c + kappa p_c) / (sum alpha + kappa); no prior => theta = p.
 *   acc[j]           : Eq. 9, Accuracy(m_j) = sum_c theta_c * recall_j(c).
 *   v                : 1 + population variance of acc over the app's models (Eq. 12 and its footnote).
 * ------------------------------------------------------------------------------------------- */
static void score_one(const orc_profiles *p, const void *feats, int64_t i, int inst, int app,
                      double *theta /* [C] scratch/out */, double *acc /* [Mmax] */, double *v)
{
    const int A = p->n_apps, C = p->n_classes, D = p->feat_dim;
    const int64_t head = ((int64_t)inst * A + app);
    const float *b = p->head_b + head * C;
    for (int c = 0; c < C; ++c) theta[c] = (double)b[c];
    for (int d = 0; d < D; ++d) {
        const double x = widen(feats, p->feat_dtype, i * D + d);
        const int64_t row = (head * D + d) * C;
        for (int c = 0; c < C; ++c) theta[c] += x * widen(p->head_w, p->feat_dtype, row + c);
    }
    double zmax = -INFINITY;
    for (int c = 0; c < C; ++c) if (theta[c] > zmax) zmax = theta[c];
    double s = 0.0;
    for (int c = 0; c < C; ++c) { theta[c] = exp(theta[c] - zmax); s += theta[c]; }
    for (int c = 0; c < C; ++c) theta[c] = theta[c] / s;
    if (p->prior_alpha) {
        const float *al = p->prior_alpha + head * C;
        double asum = 0.0;
        for (int c = 0; c < C; ++c) asum += (double)al[c];
        for (int c = 0; c < C; ++c)
            theta[c] = ((double)al[c] + p->evidence_k * theta[c]) / (asum + p->evidence_k);
    }
    const int M = p->models_per_app[app], g0 = first_model(p, app), SM = sum_models(p);
    double mean = 0.0;
    for (int j = 0; j < M; ++j) {
        const float *r = p->recall + ((int64_t)inst * SM + g0 + j) * C;
        double a = 0.0;
        for (int c = 0; c < C; ++c) a += theta[c] * (double)r[c];
        acc[j] = a;
        mean += a;
    }
    mean = mean / M;
    double var = 0.0;
    for (int j = 0; j < M; ++j) var += (acc[j] - mean) * (acc[j] - mean);
    *v = 1.0 + var / M;
}

/* Scores n requests.  acc_out [n][Mmax] (columns >= M_app are 0), v_out [n],
 * theta_out [n][C] or NULL.  Returns 0, or -1 on a bad argument. */
int orc_score(const orc_profiles *p, int64_t n, const void *feats, const int32_t *app,
              const int32_t *instance, double *acc_out, double *v_out, double *theta_out)
{
    if (!p || n < 0 || !acc_out || !v_out) return -1;
    const int C = p->n_classes, MM = max_models(p);
    int bad = 0;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        const int inst = instance ? instance[i] : 0;
        if (app[i] < 0 || app[i] >= p->n_apps || inst < 0 || inst >= p->n_instances) { bad = 1; continue; }
        double *theta = (double *)malloc(sizeof(double) * (size_t)C);
        double *acc = acc_out + i * MM;
        for (int j = 0; j < MM; ++j) acc[j] = 0.0;
        score_one(p, feats, i, inst, app[i], theta, acc, &v_out[i]);
        if (theta_out) memcpy(theta_out + i * C, theta, sizeof(double) * (size_t)C);
        free(theta);
    }
    return bad ? -1 : 0;
}

/* ---------------------------------------------------------------------------------------------
 * Penalty gamma of Eq. 2 for a request with deadline d that arrived at `arrival` and would complete at e
 * (Section 5.1).  step: 1 when the deadline is missed, else 0.  The linear and sigmoid forms are printed
 * with max(1, .) and a ratio to "d"; read literally they never fall below 1 once late, so they are read as
 *   x = (e - d) / delta,  delta = d - arrival (the relative deadline),
 *   linear : gamma = min(max(x, 0), 1)
 *   sigmoid: gamma = 0 for x <= 0, 1 for x >= 1, else 1 / (1 + ((1 - x) / x)^3)
 * so that the utility degrades from the deadline on and is gone once the request is late by its whole relative
 * deadline.  A request whose deadline is not after its arrival falls back to the step form.
 * ------------------------------------------------------------------------------------------- */
double orc_penalty(int kind, int64_t d, int64_t arrival, int64_t e)
{
    const int64_t delta = d - arrival;
    if (kind == ORC_PEN_STEP || delta <= 0) return d < e ? 1.0 : 0.0;
    if (e <= d) return 0.0;
    if (e - d >= delta) return 1.0;
    const double x = (double)(e - d) / (double)delta;
    if (kind == ORC_PEN_LINEAR) return x;
    const double r = (1.0 - x) / x;
    return 1.0 / (1.0 + r * r * r);
}

/* A request is hopeless when even the earliest completion `emin` its group can reach leaves it no utility:
 * gamma = 1 there.  Stated on the integer times, not on the rounded value of gamma: under the step penalty the
 * deadline precedes emin; under the soft penalties x >= 1, i.e. emin is at least the whole relative deadline
 * after the deadline (the sigmoid expression rounds to 1.0 in fp64 slightly before x reaches 1; such a request
 * is not hopeless yet, it merely earns nothing if served then). */
static int hopeless(int kind, int64_t d, int64_t arrival, int64_t emin)
{
    const int64_t delta = d - arrival;
    if (kind == ORC_PEN_STEP || delta <= 0) return d < emin;
    return emin - d >= delta;
}

/* ---------------------------------------------------------------------------------------------
 * Scheduling rounds of one instance (Section 4.2: groups = applications, Eq. 14 group priority,
 * Eq. 13 applied to the group with summed member utilities (Eq. 2), Algorithm 1's greedy branch
 * taken one batch at a time).  Readings of points the paper leaves open:
 *   - inside a group requests are taken in (deadline, id) order;
 *   - a candidate is (model m, allowed batch size b): the first b' = min(b, n_a) live requests
 *     of the group run as one batch that completes at e = T + swap_m*[m != loaded] + alpha_m
 *     + beta_m*b' (Eq. 1 with the swap time kept separate from the inference latency);
 *   - a member contributes acc[member][m] * (1 - gamma) with the application's penalty gamma of
 *     orc_penalty() (step penalty: 0 when its deadline < e, else acc[member][m]);
 *   - a request at the head of its group's queue whose penalty is already 1 at the earliest
 *     completion any candidate of the group could reach from the current state can never earn
 *     utility: it is retired as EXPIRED (for the step penalty: every request with deadline < that time);
 *   - group priorities are re-evaluated every round over the live members, with d measured
 *     from the current clock in seconds and scaled by tau;
 *   - ties: lowest application index; lowest model index, then smallest batch size.
 * ------------------------------------------------------------------------------------------- */
typedef struct { int64_t deadline, id; } qkey;

static int cmp_qkey(const void *x, const void *y)
{
    const qkey *a = (const qkey *)x, *b = (const qkey *)y;
    if (a->deadline != b->deadline) return a->deadline < b->deadline ? -1 : 1;
    if (a->id != b->id) return a->id < b->id ? -1 : 1;
    return 0;
}

typedef struct { int64_t arrival, id; } akey;

static int cmp_akey(const void *x, const void *y)
{
    const akey *a = (const akey *)x, *b = (const akey *)y;
    if (a->arrival != b->arrival) return a->arrival < b->arrival ? -1 : 1;
    if (a->id != b->id) return a->id < b->id ? -1 : 1;
    return 0;
}

static void drain_instance(const orc_profiles *p, int inst, int64_t lo, int64_t hi,
                           const int32_t *app, const int64_t *arrival, const int64_t *deadline,
                           const double *acc, const double *v, int64_t t0, int32_t loaded0,
                           int trace_mode, int64_t max_rounds, orc_round_rec *rounds, int64_t cap,
                           int64_t *n_rounds, orc_req_rec *reqs, int64_t *t_end, int32_t *loaded_end)
{
    const int A = p->n_apps, MM = max_models(p), SM = sum_models(p), nB = p->n_batch_sizes;
    const int64_t *al = p->lat_alpha_ns + (int64_t)inst * SM;
    const int64_t *be = p->lat_beta_ns + (int64_t)inst * SM;
    const int64_t *sw = p->swap_ns + (int64_t)inst * SM;
    const int64_t n = hi - lo;
    const double tau = p->prio_time_scale_s;

    akey *arr = (akey *)malloc(sizeof(akey) * (size_t)(n > 0 ? n : 1));
    for (int64_t i = 0; i < n; ++i) { arr[i].arrival = arrival[lo + i]; arr[i].id = lo + i; }
    qsort(arr, (size_t)n, sizeof(akey), cmp_akey);
    qkey **q = (qkey **)malloc(sizeof(qkey *) * (size_t)A);
    int64_t *head = (int64_t *)calloc((size_t)A, sizeof(int64_t));
    int64_t *tail = (int64_t *)calloc((size_t)A, sizeof(int64_t));
    for (int a = 0; a < A; ++a) q[a] = (qkey *)malloc(sizeof(qkey) * (size_t)(n > 0 ? n : 1));
    for (int64_t i = lo; i < hi; ++i) {
        reqs[i].status = ORC_PENDING; reqs[i].round = -1; reqs[i].model = -1; reqs[i].pad_ = 0; reqs[i].order = 0;
    }

    int64_t T = t0, ap = 0, round = 0, next_order = 1;
    int32_t L = loaded0, exp_since = 0;
    while (round < max_rounds) {
        /* 1. requests that have arrived join their application's group */
        int inserted = 0;
        while (ap < n && (!trace_mode || arr[ap].arrival <= T)) {
            const int64_t id = arr[ap].id;
            const int a = app[id];
            q[a][tail[a]].deadline = deadline[id];
            q[a][tail[a]].id = id;
            ++tail[a]; ++ap; inserted = 1;
        }
        int64_t live = 0;
        for (int a = 0; a < A; ++a) live += tail[a] - head[a];
        if (live == 0) {
            if (ap < n) { T = arr[ap].arrival; continue; }
            break;
        }
        /* 2. order inside each group */
        if (inserted)
            for (int a = 0; a < A; ++a)
                qsort(q[a] + head[a], (size_t)(tail[a] - head[a]), sizeof(qkey), cmp_qkey);
        /* 3. retire requests that no candidate of their group can complete in time */
        const int64_t bmin = p->batch_sizes[0];
        for (int a = 0; a < A; ++a) {
            const int g0 = first_model(p, a), M = p->models_per_app[a];
            int64_t emin = INT64_MAX;
            for (int j = 0; j < M; ++j) {
                const int g = g0 + j;
                const int64_t e = T + (g != L ? sw[g] : 0) + al[g] + be[g] * bmin;
                if (e < emin) emin = e;
            }
            const int pk = p->penalty_kind ? p->penalty_kind[a] : ORC_PEN_STEP;
            while (head[a] < tail[a] && hopeless(pk, q[a][head[a]].deadline, arrival[q[a][head[a]].id], emin)) {
                orc_req_rec *r = &reqs[q[a][head[a]].id];
                r->status = ORC_EXPIRED; r->round = (int32_t)round;
                ++head[a]; ++exp_since;
            }
        }
        live = 0;
        for (int a = 0; a < A; ++a) live += tail[a] - head[a];
        if (live == 0) continue;
        /* 4. group priority, Eq. 14 over Eq. 12 */
        int best_a = -1;
        double best_p = 0.0, second_p = -INFINITY;
        for (int a = 0; a < A; ++a) {
            const int64_t na = tail[a] - head[a];
            if (na == 0) continue;
            double s = 0.0;
            for (int64_t k = head[a]; k < tail[a]; ++k) {
                const double dt = (double)(q[a][k].deadline - T) * 1e-9 / tau;
                s += v[q[a][k].id] * exp(-dt);
            }
            const double pr = s / (double)na;
            if (best_a < 0) { best_a = a; best_p = pr; }
            else if (pr > best_p) { second_p = best_p; best_a = a; best_p = pr; }
            else if (pr < best_p && pr > second_p) second_p = pr;
        }
        /* 5./6. every (model, batch size) candidate of the chosen group; best summed utility */
        const int a = best_a, g0 = first_model(p, a), M = p->models_per_app[a];
        const int64_t na = tail[a] - head[a];
        const int pen = p->penalty_kind ? p->penalty_kind[a] : ORC_PEN_STEP;
        int best_j = -1, best_b = 0;
        int64_t best_bp = 0, best_e = 0;
        double best_u = 0.0, second_u = -INFINITY;
        for (int j = 0; j < M; ++j) {
            const int g = g0 + j;
            for (int bi = 0; bi < nB; ++bi) {
                const int64_t b = p->batch_sizes[bi], bp = b < na ? b : na;
                const int64_t e = T + (g != L ? sw[g] : 0) + al[g] + be[g] * bp;
                double u = 0.0;
                for (int64_t k = 0; k < bp; ++k) {
                    const qkey *m = &q[a][head[a] + k];
                    if (pen == ORC_PEN_STEP) { if (!(m->deadline < e)) u += acc[m->id * MM + j]; }
                    else u += acc[m->id * MM + j] * (1.0 - orc_penalty(pen, m->deadline, arrival[m->id], e));
                }
                if (best_j < 0) { best_j = j; best_b = (int)b; best_bp = bp; best_e = e; best_u = u; }
                else if (u > best_u) { second_u = best_u; best_j = j; best_b = (int)b; best_bp = bp; best_e = e; best_u = u; }
                else if (u < best_u && u > second_u) second_u = u;
            }
        }
        /* 7. emit the batch, remove its members, advance the clock, remember the loaded model */
        for (int64_t k = 0; k < best_bp; ++k) {
            orc_req_rec *r = &reqs[q[a][head[a] + k].id];
            r->status = ORC_SCHEDULED; r->round = (int32_t)round; r->model = g0 + best_j; r->order = next_order++;
        }
        head[a] += best_bp;
        if (rounds && round < cap) {
            orc_round_rec *rr = &rounds[round];
            rr->instance = inst; rr->round = (int32_t)round; rr->app = a; rr->model = g0 + best_j;
            rr->batch = best_b; rr->n_members = (int32_t)best_bp; rr->n_expired = exp_since; rr->pad_ = 0;
            rr->t_start_ns = T; rr->t_end_ns = best_e; rr->utility = best_u; rr->group_priority = best_p;
            rr->util_margin = (second_u == -INFINITY || !(best_u > 0.0)) ? INFINITY : (best_u - second_u) / best_u;
            rr->prio_margin = (second_p == -INFINITY || !(best_p > 0.0)) ? INFINITY : (best_p - second_p) / best_p;
        }
        exp_since = 0;
        T = best_e; L = g0 + best_j; ++round;
    }
    *n_rounds = round; *t_end = T; *loaded_end = L;
    for (int a = 0; a < A; ++a) free(q[a]);
    free(q); free(head); free(tail); free(arr);
}

/* Runs up to max_rounds rounds of every instance.  Requests must be grouped by instance in
 * ascending order (instance == NULL means one instance).  rounds [I][cap] (may be NULL),
 * n_rounds [I], reqs [n], t_end [I], loaded_end [I].  Returns 0, -1 on a bad argument. */
int orc_drain(const orc_profiles *p, int64_t n, const int32_t *app, const int32_t *instance,
              const int64_t *arrival, const int64_t *deadline, const double *acc, const double *v,
              const int64_t *t0, const int32_t *loaded0, int trace_mode, int64_t max_rounds,
              orc_round_rec *rounds, int64_t cap, int64_t *n_rounds, orc_req_rec *reqs,
              int64_t *t_end, int32_t *loaded_end)
{
    if (!p || n < 0 || !n_rounds || !reqs || !t_end || !loaded_end) return -1;
    const int I = p->n_instances;
    int64_t *start = (int64_t *)malloc(sizeof(int64_t) * (size_t)(I + 1));
    {
        int64_t i = 0;
        for (int k = 0; k < I; ++k) {
            start[k] = i;
            while (i < n && (instance ? instance[i] : 0) == k) ++i;
        }
        start[I] = i;
        if (i != n) { free(start); return -1; }
    }
#pragma omp parallel for schedule(dynamic, 1)
    for (int k = 0; k < I; ++k)
        drain_instance(p, k, start[k], start[k + 1], app, arrival, deadline, acc, v, t0[k], loaded0[k],
                       trace_mode, max_rounds, rounds ? rounds + (int64_t)k * cap : NULL, cap,
                       &n_rounds[k], reqs, &t_end[k], &loaded_end[k]);
    free(start);
    return 0;
}

/* Number of threads the parallel loops above use. */
int orc_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
