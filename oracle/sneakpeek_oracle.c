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
 * and monotonicity).  Also readings: which requests form a data-aware sub-group (orc_score's label), how a whole
 * group is run in the exhaustive branch of Algorithm 1 (orc_bruteforce), what "max accuracy" picks when no model
 * meets the deadline (orc_baseline); each is stated where it is implemented.
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
    int32_t instance, round, app, model, batch, n_members, n_expired;
    int32_t label;        /* sub-group of the application that was served: predicted label, -1 = not split / inconclusive */
    int32_t worker, pad_; /* worker that ran the batch (0 with a single worker) */
    int64_t t_start_ns, t_end_ns;
    double utility, group_priority;
    double util_margin;   /* (U1-U2)/U1 over candidates of the chosen group with a different value; +inf if none */
    double prio_margin;   /* (P1-P2)/P1 over the other non-empty groups; +inf if none */
} orc_round_rec;

typedef struct {
    int32_t status, round, model;
    int32_t worker;       /* worker the request ran on (0 with a single worker) */
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
                      double *theta /* [C] scratch/out */, double *acc /* [Mmax] */, double *v, int32_t *label)
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
    /* Data-aware sub-group ("Enhancements for Grouped Scheduling", Section 4.3): the request belongs to the sub-group
     * of label c when theta_c > 0.5 (at most one label can), and stays with its application's unsplit remainder when
     * every theta_c <= 0.5. */
    if (label) {
        *label = -1;
        for (int c = 0; c < C; ++c) if (theta[c] > 0.5) *label = c;
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
 * theta_out [n][C] or NULL, label_out [n] or NULL (predicted label, -1 = inconclusive).
 * Returns 0, or -1 on a bad argument. */
int orc_score(const orc_profiles *p, int64_t n, const void *feats, const int32_t *app,
              const int32_t *instance, double *acc_out, double *v_out, double *theta_out, int32_t *label_out)
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
        score_one(p, feats, i, inst, app[i], theta, acc, &v_out[i], label_out ? &label_out[i] : NULL);
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
                           const int32_t *app, const int32_t *label, const int64_t *arrival, const int64_t *deadline,
                           const double *acc, const double *v, int64_t t0, int32_t loaded0,
                           int trace_mode, int64_t max_rounds, orc_round_rec *rounds, int64_t cap,
                           int64_t *n_rounds, orc_req_rec *reqs, int64_t *t_end, int32_t *loaded_end)
{
    /* Groups: the applications (Section 4.2), or, with labels given, the data-aware sub-groups of Section 4.3: group
     * index = app * (C + 1) + label + 1, so an application's unsplit remainder (label -1) comes before its per-label
     * sub-groups and "lowest application" generalises to "lowest group index".  GW = groups per application. */
    const int GW = label ? p->n_classes + 1 : 1;
    const int A = p->n_apps * GW, MM = max_models(p), SM = sum_models(p), nB = p->n_batch_sizes;
#define GROUP_OF(id) (app[id] * GW + (label ? label[id] + 1 : 0))
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
    for (int64_t i = lo; i < hi; ++i) ++tail[GROUP_OF(i)];              /* group sizes, to size the queues */
    for (int a = 0; a < A; ++a) { q[a] = (qkey *)malloc(sizeof(qkey) * (size_t)(tail[a] > 0 ? tail[a] : 1)); tail[a] = 0; }
    for (int64_t i = lo; i < hi; ++i) {
        reqs[i].status = ORC_PENDING; reqs[i].round = -1; reqs[i].model = -1; reqs[i].worker = 0; reqs[i].order = 0;
    }

    int64_t T = t0, ap = 0, round = 0, next_order = 1;
    int32_t L = loaded0, exp_since = 0;
    while (round < max_rounds) {
        /* 1. requests that have arrived join their application's group */
        int inserted = 0;
        while (ap < n && (!trace_mode || arr[ap].arrival <= T)) {
            const int64_t id = arr[ap].id;
            const int a = GROUP_OF(id);
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
            if (head[a] == tail[a]) continue;
            const int g0 = first_model(p, a / GW), M = p->models_per_app[a / GW];
            int64_t emin = INT64_MAX;
            for (int j = 0; j < M; ++j) {
                const int g = g0 + j;
                const int64_t e = T + (g != L ? sw[g] : 0) + al[g] + be[g] * bmin;
                if (e < emin) emin = e;
            }
            const int pk = p->penalty_kind ? p->penalty_kind[a / GW] : ORC_PEN_STEP;
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
        const int a = best_a, g0 = first_model(p, a / GW), M = p->models_per_app[a / GW];
        const int64_t na = tail[a] - head[a];
        const int pen = p->penalty_kind ? p->penalty_kind[a / GW] : ORC_PEN_STEP;
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
            rr->instance = inst; rr->round = (int32_t)round; rr->app = a / GW; rr->model = g0 + best_j;
            rr->batch = best_b; rr->n_members = (int32_t)best_bp; rr->n_expired = exp_since;
            rr->label = label ? a % GW - 1 : -1; rr->worker = 0; rr->pad_ = 0;
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
#undef GROUP_OF
}

/* Runs up to max_rounds rounds of every instance.  Requests must be grouped by instance in
 * ascending order (instance == NULL means one instance).  label: predicted labels from orc_score() to schedule the
 * data-aware sub-groups of Section 4.3, or NULL to schedule whole applications.  rounds [I][cap] (may be NULL),
 * n_rounds [I], reqs [n], t_end [I], loaded_end [I].  Returns 0, -1 on a bad argument. */
int orc_drain(const orc_profiles *p, int64_t n, const int32_t *app, const int32_t *instance, const int32_t *label,
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
        drain_instance(p, k, start[k], start[k + 1], app, label, arrival, deadline, acc, v, t0[k], loaded0[k],
                       trace_mode, max_rounds, rounds ? rounds + (int64_t)k * cap : NULL, cap,
                       &n_rounds[k], reqs, &t_end[k], &loaded_end[k]);
    free(start);
    return 0;
}


/* ---------------------------------------------------------------------------------------------
 * Exhaustive branch of Algorithm 1 (Section 4.2: when the number of groups is at most the threshold tau, the
 * group-level problem is solved exactly).  A solution is an order of the non-empty groups and one model per group;
 * every group is served whole, on its model, before the next group starts.  Reading of "served whole" under batch
 * sizes: the group's members, in (deadline, id) order, run back to back in batches of the largest allowed size (the
 * last batch takes the remainder); batch k completes at e = T + swap*[model != loaded] + alpha + beta*b' (Eq. 1) and
 * each member earns acc * (1 - gamma) (Eq. 2).  Nothing is retired: every request gets a model and an order (Eq. 5).
 * All G! * prod M_g solutions are evaluated; the best total (Eq. 3's sum) wins, the first in enumeration order on a
 * tie: orders in lexicographic order of the group indices, then model choices in lexicographic order with the
 * lowest group index as the slowest digit.  One instance (instance 0 of the profiles); groups as in drain_instance.
 * Returns 0, -1 on a bad argument, -2 when there are more than 8 non-empty groups or more than 2^31 solutions.
 * ------------------------------------------------------------------------------------------- */
typedef struct { int g, M, g0, pen; int64_t n; qkey *q; } bf_group;

static double bf_eval(const orc_profiles *p, const bf_group *grp, int G, const int *perm, const int *choice,
                      const int64_t *arrival, const double *acc, int MM, int64_t t0, int32_t loaded0,
                      orc_round_rec *rounds, int64_t cap, int64_t *n_rounds, orc_req_rec *reqs, int64_t *t_end, int32_t *l_end)
{
    const int64_t *al = p->lat_alpha_ns, *be = p->lat_beta_ns, *sw = p->swap_ns;
    const int64_t bmax = p->batch_sizes[p->n_batch_sizes - 1];
    int64_t T = t0, order = 1, round = 0;
    int32_t L = loaded0;
    double total = 0.0;
    for (int pos = 0; pos < G; ++pos) {
        const bf_group *gr = &grp[perm[pos]];
        const int j = choice[perm[pos]], m = gr->g0 + j;
        for (int64_t k0 = 0; k0 < gr->n; k0 += bmax) {
            const int64_t bp = gr->n - k0 < bmax ? gr->n - k0 : bmax;
            const int64_t e = T + (m != L ? sw[m] : 0) + al[m] + be[m] * bp;
            double u = 0.0;
            for (int64_t k = 0; k < bp; ++k) {
                const qkey *mem = &gr->q[k0 + k];
                const double contrib = acc[mem->id * MM + j] * (1.0 - orc_penalty(gr->pen, mem->deadline, arrival[mem->id], e));
                u += contrib;
                total += contrib;
                if (reqs) {
                    orc_req_rec *r = &reqs[mem->id];
                    r->status = ORC_SCHEDULED; r->round = (int32_t)round; r->model = m; r->worker = 0; r->order = order++;
                }
            }
            if (rounds && round < cap) {
                orc_round_rec *rr = &rounds[round];
                memset(rr, 0, sizeof *rr);
                rr->instance = 0; rr->round = (int32_t)round; rr->app = 0; rr->model = m;
                rr->batch = (int32_t)bmax; rr->n_members = (int32_t)bp; rr->t_start_ns = T; rr->t_end_ns = e; rr->utility = u;
                rr->util_margin = INFINITY; rr->prio_margin = INFINITY;
            }
            T = e; L = m; ++round;
        }
    }
    if (n_rounds) *n_rounds = round;
    if (t_end) *t_end = T;
    if (l_end) *l_end = L;
    return total;
}

static int bf_next_perm(int *a, int n)
{
    int i = n - 2;
    while (i >= 0 && a[i] > a[i + 1]) --i;
    if (i < 0) return 0;
    int j = n - 1;
    while (a[j] < a[i]) --j;
    int t = a[i]; a[i] = a[j]; a[j] = t;
    for (int l = i + 1, r = n - 1; l < r; ++l, --r) { t = a[l]; a[l] = a[r]; a[r] = t; }
    return 1;
}

int orc_bruteforce(const orc_profiles *p, int64_t n, const int32_t *app, const int32_t *label, const int64_t *arrival,
                   const int64_t *deadline, const double *acc, int64_t t0, int32_t loaded0, orc_round_rec *rounds,
                   int64_t cap, int64_t *n_rounds, orc_req_rec *reqs, int64_t *t_end, int32_t *loaded_end,
                   double *best_total, double *second_total, int64_t *n_solutions)
{
    if (!p || n < 0 || !n_rounds || !reqs || !t_end || !loaded_end || !best_total || !n_solutions) return -1;
    const int GW = label ? p->n_classes + 1 : 1, NG = p->n_apps * GW, MM = max_models(p);
    int64_t *count = (int64_t *)calloc((size_t)NG, sizeof(int64_t));
    for (int64_t i = 0; i < n; ++i) ++count[app[i] * GW + (label ? label[i] + 1 : 0)];
    bf_group grp[8];
    int G = 0;
    for (int g = 0; g < NG; ++g) {
        if (!count[g]) continue;
        if (G == 8) { free(count); return -2; }
        grp[G].g = g; grp[G].M = p->models_per_app[g / GW]; grp[G].g0 = first_model(p, g / GW);
        grp[G].pen = p->penalty_kind ? p->penalty_kind[g / GW] : ORC_PEN_STEP;
        grp[G].n = 0; grp[G].q = (qkey *)malloc(sizeof(qkey) * (size_t)count[g]);
        ++G;
    }
    for (int64_t i = 0; i < n; ++i) {
        const int g = app[i] * GW + (label ? label[i] + 1 : 0);
        for (int k = 0; k < G; ++k)
            if (grp[k].g == g) { grp[k].q[grp[k].n].deadline = deadline[i]; grp[k].q[grp[k].n].id = i; ++grp[k].n; }
    }
    double n_sol = 1.0;
    for (int k = 0; k < G; ++k) { qsort(grp[k].q, (size_t)grp[k].n, sizeof(qkey), cmp_qkey); n_sol *= (double)grp[k].M * (double)(k + 1); }
    int rc = 0;
    if (n_sol > 2147483648.0) rc = -2;
    int perm[8], choice[8], best_perm[8], best_choice[8];
    double best = -INFINITY, second = -INFINITY;
    int64_t visited = 0;
    if (rc == 0) {
        for (int k = 0; k < G; ++k) perm[k] = k;
        do {
            for (int k = 0; k < G; ++k) choice[k] = 0;
            for (;;) {
                const double tot = bf_eval(p, grp, G, perm, choice, arrival, acc, MM, t0, loaded0, NULL, 0, NULL, NULL, NULL, NULL);
                ++visited;
                if (tot > best) { second = best; best = tot; memcpy(best_perm, perm, sizeof perm); memcpy(best_choice, choice, sizeof choice); }
                else if (tot < best && tot > second) second = tot;
                int k = G - 1;                                   /* next model tuple: last group is the fastest digit */
                while (k >= 0 && ++choice[k] == grp[k].M) { choice[k] = 0; --k; }
                if (k < 0) break;
            }
        } while (bf_next_perm(perm, G));
        for (int64_t i = 0; i < n; ++i) { reqs[i].status = ORC_PENDING; reqs[i].round = -1; reqs[i].model = -1; reqs[i].worker = 0; reqs[i].order = 0; }
        if (G > 0) {
            bf_eval(p, grp, G, best_perm, best_choice, arrival, acc, MM, t0, loaded0, rounds, cap, n_rounds, reqs, t_end, loaded_end);
            if (rounds) {                                        /* application and label of every emitted batch */
                int64_t r = 0;
                const int64_t bmax = p->batch_sizes[p->n_batch_sizes - 1];
                for (int pos = 0; pos < G; ++pos)
                    for (int64_t k0 = 0; k0 < grp[best_perm[pos]].n; k0 += bmax, ++r)
                        if (r < cap) { rounds[r].app = grp[best_perm[pos]].g / GW; rounds[r].label = label ? grp[best_perm[pos]].g % GW - 1 : -1; }
            }
        } else { *n_rounds = 0; *t_end = t0; *loaded_end = loaded0; }
        *best_total = G > 0 ? best : 0.0;
        if (second_total) *second_total = second;
        *n_solutions = visited;
    }
    for (int k = 0; k < G; ++k) free(grp[k].q);
    free(count);
    return rc;
}

/* ---------------------------------------------------------------------------------------------
 * Request-level baselines of the evaluation (Section 5.1, "Baselines and Metrics"): an ordering policy plus a
 * per-request model selection, one request at a time (batch size 1), nothing retired.
 *   order  EDF: (deadline, id) ascending.  Priority: Eq. 12, v_i * exp(-(d_i - t0)/tau) descending, then id
 *          (a common clock shift rescales every priority alike, so the order does not change while the schedule runs).
 *   model  Locally optimal (Eq. 13): the model with the highest utility acc * (1 - gamma(d, e)) at the time the
 *          request starts, e = T + swap*[model != loaded] + alpha + beta.  Max accuracy: the most accurate model that
 *          still meets the deadline (d >= e); reading for the case the paper leaves open: when none meets it, the most
 *          accurate model of all.  Ties: lowest model.
 * policy 0 = MaxAcc-EDF, 1 = LO-EDF, 2 = LO-Priority.  min_margin [I]: smallest relative gap met in an instance
 * between the winning and the runner-up score of a decision, and between consecutive priorities of the order.
 * ------------------------------------------------------------------------------------------- */
typedef struct { double prio; int64_t deadline, id; } bkey;
static int cmp_b_edf(const void *x, const void *y)
{
    const bkey *a = (const bkey *)x, *b = (const bkey *)y;
    if (a->deadline != b->deadline) return a->deadline < b->deadline ? -1 : 1;
    return a->id < b->id ? -1 : a->id > b->id;
}
static int cmp_b_prio(const void *x, const void *y)
{
    const bkey *a = (const bkey *)x, *b = (const bkey *)y;
    if (a->prio != b->prio) return a->prio > b->prio ? -1 : 1;
    return a->id < b->id ? -1 : a->id > b->id;
}

int orc_baseline(const orc_profiles *p, int policy, int64_t n, const int32_t *app, const int32_t *instance,
                 const int64_t *arrival, const int64_t *deadline, const double *acc, const double *v,
                 const int64_t *t0, const int32_t *loaded0, orc_round_rec *rounds, int64_t cap, int64_t *n_rounds,
                 orc_req_rec *reqs, int64_t *t_end, int32_t *loaded_end, double *min_margin)
{
    if (!p || n < 0 || policy < 0 || policy > 2 || !n_rounds || !reqs || !t_end || !loaded_end) return -1;
    const int I = p->n_instances, MM = max_models(p), SM = sum_models(p);
    int64_t *start = (int64_t *)malloc(sizeof(int64_t) * (size_t)(I + 1));
    {
        int64_t i = 0;
        for (int k = 0; k < I; ++k) { start[k] = i; while (i < n && (instance ? instance[i] : 0) == k) ++i; }
        start[I] = i;
        if (i != n) { free(start); return -1; }
    }
#pragma omp parallel for schedule(dynamic, 1)
    for (int inst = 0; inst < I; ++inst) {
        const int64_t lo = start[inst], m = start[inst + 1] - lo;
        const int64_t *al = p->lat_alpha_ns + (int64_t)inst * SM, *be = p->lat_beta_ns + (int64_t)inst * SM;
        const int64_t *sw = p->swap_ns + (int64_t)inst * SM;
        bkey *ord = (bkey *)malloc(sizeof(bkey) * (size_t)(m > 0 ? m : 1));
        double margin = INFINITY;
        for (int64_t k = 0; k < m; ++k) {
            const int64_t id = lo + k;
            ord[k].id = id; ord[k].deadline = deadline[id];
            ord[k].prio = v[id] * exp(-((double)(deadline[id] - t0[inst]) * 1e-9 / p->prio_time_scale_s));
        }
        qsort(ord, (size_t)m, sizeof(bkey), policy == 2 ? cmp_b_prio : cmp_b_edf);
        if (policy == 2)
            for (int64_t k = 0; k + 1 < m; ++k)
                if (ord[k].prio > ord[k + 1].prio && ord[k].prio > 0.0) {
                    const double g = (ord[k].prio - ord[k + 1].prio) / ord[k].prio;
                    if (g < margin) margin = g;
                }
        int64_t T = t0[inst];
        int32_t L = loaded0[inst];
        for (int64_t k = 0; k < m; ++k) {
            const int64_t id = ord[k].id;
            const int a = app[id], g0 = first_model(p, a), M = p->models_per_app[a];
            const int pen = p->penalty_kind ? p->penalty_kind[a] : ORC_PEN_STEP;
            int best = -1, any_feasible = 0;
            double best_s = -INFINITY, second_s = -INFINITY;
            if (policy == 0)
                for (int j = 0; j < M; ++j) {
                    const int g = g0 + j;
                    if (!(deadline[id] < T + (g != L ? sw[g] : 0) + al[g] + be[g])) any_feasible = 1;
                }
            for (int j = 0; j < M; ++j) {
                const int g = g0 + j;
                const int64_t e = T + (g != L ? sw[g] : 0) + al[g] + be[g];
                double sc;
                if (policy == 0) {
                    if (any_feasible && deadline[id] < e) continue;
                    sc = acc[id * MM + j];
                } else sc = acc[id * MM + j] * (1.0 - orc_penalty(pen, deadline[id], arrival[id], e));
                if (best < 0 || sc > best_s) { if (best >= 0) second_s = best_s; best = j; best_s = sc; }
                else if (sc < best_s && sc > second_s) second_s = sc;
            }
            if (second_s != -INFINITY && best_s > 0.0 && (best_s - second_s) / best_s < margin) margin = (best_s - second_s) / best_s;
            const int g = g0 + best;
            const int64_t e = T + (g != L ? sw[g] : 0) + al[g] + be[g];
            const double u = acc[id * MM + best] * (1.0 - orc_penalty(pen, deadline[id], arrival[id], e));
            orc_req_rec *r = &reqs[id];
            r->status = ORC_SCHEDULED; r->round = (int32_t)k; r->model = g; r->worker = 0; r->order = k + 1;
            if (rounds && k < cap) {
                orc_round_rec *rr = &rounds[(int64_t)inst * cap + k];
                memset(rr, 0, sizeof *rr);
                rr->instance = inst; rr->round = (int32_t)k; rr->app = a; rr->model = g; rr->batch = 1; rr->n_members = 1;
                rr->label = -1; rr->t_start_ns = T; rr->t_end_ns = e; rr->utility = u; rr->group_priority = ord[k].prio;
                rr->util_margin = INFINITY; rr->prio_margin = INFINITY;
            }
            T = e; L = g;
        }
        n_rounds[inst] = m; t_end[inst] = T; loaded_end[inst] = L;
        if (min_margin) min_margin[inst] = margin;
        free(ord);
    }
    free(start);
    return 0;
}


/* ---------------------------------------------------------------------------------------------
 * Several workers (Section 6: the schedule gains a worker index and every model variant has a latency profile per
 * worker; the objective is Eq. 15, the same summed utility).  The paper states the objective only; the reading taken
 * here is list scheduling with the single-worker round: worker k has its own clock T_k and resident model L_k; the
 * worker that is free first (lowest T_k, then lowest k) takes the next batch at T = T_k, chosen exactly as in
 * drain_instance (arrivals up to T join, hopeless requests leave, the group with the highest Eq. 14 priority at T is
 * served by its best (model, batch size) candidate ON THAT WORKER), and its clock moves to the batch's completion.
 * A request is hopeless when no worker could complete it in time: emin = min over workers and models of
 * T_k + swap*[model != L_k] + alpha + beta*b_min.  The largest allowed batch size is the maximum group size the
 * Discussion asks for.  When nothing is pending, every idle worker's clock moves to the next arrival.
 * Profiles: lat_alpha_ns / lat_beta_ns / swap_ns of `p` are read as [W][sumM] (worker-major); one instance.
 * With W = 1 this is drain_instance.
 * ------------------------------------------------------------------------------------------- */
int orc_drain_workers(const orc_profiles *p, int W, int64_t n, const int32_t *app, const int32_t *label,
                      const int64_t *arrival, const int64_t *deadline, const double *acc, const double *v, int64_t t0,
                      int32_t loaded0, int trace_mode, int64_t max_rounds, orc_round_rec *rounds, int64_t cap,
                      int64_t *n_rounds, orc_req_rec *reqs, int64_t *t_end /* [W] */, int32_t *loaded_end /* [W] */)
{
    if (!p || W < 1 || n < 0 || !n_rounds || !reqs || !t_end || !loaded_end) return -1;
    const int GW = label ? p->n_classes + 1 : 1;
    const int A = p->n_apps * GW, MM = max_models(p), SM = sum_models(p), nB = p->n_batch_sizes;
    const double tau = p->prio_time_scale_s;
#define GROUP_OF(id) (app[id] * GW + (label ? label[id] + 1 : 0))
    akey *arr = (akey *)malloc(sizeof(akey) * (size_t)(n > 0 ? n : 1));
    for (int64_t i = 0; i < n; ++i) { arr[i].arrival = arrival[i]; arr[i].id = i; }
    qsort(arr, (size_t)n, sizeof(akey), cmp_akey);
    qkey **q = (qkey **)malloc(sizeof(qkey *) * (size_t)A);
    int64_t *head = (int64_t *)calloc((size_t)A, sizeof(int64_t));
    int64_t *tail = (int64_t *)calloc((size_t)A, sizeof(int64_t));
    for (int64_t i = 0; i < n; ++i) ++tail[GROUP_OF(i)];
    for (int a = 0; a < A; ++a) { q[a] = (qkey *)malloc(sizeof(qkey) * (size_t)(tail[a] > 0 ? tail[a] : 1)); tail[a] = 0; }
    for (int64_t i = 0; i < n; ++i) { reqs[i].status = ORC_PENDING; reqs[i].round = -1; reqs[i].model = -1; reqs[i].worker = 0; reqs[i].order = 0; }
    for (int k = 0; k < W; ++k) { t_end[k] = t0; loaded_end[k] = loaded0; }
    int64_t ap = 0, round = 0, next_order = 1;
    int32_t exp_since = 0;
    while (round < max_rounds) {
        int wk = 0;                                            /* the worker that is free first */
        for (int k = 1; k < W; ++k) if (t_end[k] < t_end[wk]) wk = k;
        const int64_t T = t_end[wk];
        const int32_t L = loaded_end[wk];
        const int64_t *al = p->lat_alpha_ns + (int64_t)wk * SM, *be = p->lat_beta_ns + (int64_t)wk * SM, *sw = p->swap_ns + (int64_t)wk * SM;
        int inserted = 0;
        while (ap < n && (!trace_mode || arr[ap].arrival <= T)) {
            const int64_t id = arr[ap].id;
            const int a = GROUP_OF(id);
            q[a][tail[a]].deadline = deadline[id]; q[a][tail[a]].id = id;
            ++tail[a]; ++ap; inserted = 1;
        }
        int64_t live = 0;
        for (int a = 0; a < A; ++a) live += tail[a] - head[a];
        if (live == 0) {
            if (ap < n) { for (int k = 0; k < W; ++k) if (t_end[k] < arr[ap].arrival) t_end[k] = arr[ap].arrival; continue; }
            break;
        }
        if (inserted)
            for (int a = 0; a < A; ++a) qsort(q[a] + head[a], (size_t)(tail[a] - head[a]), sizeof(qkey), cmp_qkey);
        const int64_t bmin = p->batch_sizes[0];
        for (int a = 0; a < A; ++a) {
            if (head[a] == tail[a]) continue;
            const int g0 = first_model(p, a / GW), M = p->models_per_app[a / GW];
            int64_t emin = INT64_MAX;
            for (int k = 0; k < W; ++k)
                for (int j = 0; j < M; ++j) {
                    const int g = g0 + j;
                    const int64_t e = t_end[k] + (g != loaded_end[k] ? p->swap_ns[(int64_t)k * SM + g] : 0) +
                                      p->lat_alpha_ns[(int64_t)k * SM + g] + p->lat_beta_ns[(int64_t)k * SM + g] * bmin;
                    if (e < emin) emin = e;
                }
            const int pk = p->penalty_kind ? p->penalty_kind[a / GW] : ORC_PEN_STEP;
            while (head[a] < tail[a] && hopeless(pk, q[a][head[a]].deadline, arrival[q[a][head[a]].id], emin)) {
                orc_req_rec *r = &reqs[q[a][head[a]].id];
                r->status = ORC_EXPIRED; r->round = (int32_t)round;
                ++head[a]; ++exp_since;
            }
        }
        live = 0;
        for (int a = 0; a < A; ++a) live += tail[a] - head[a];
        if (live == 0) continue;
        int best_a = -1;
        double best_p = 0.0, second_p = -INFINITY;
        for (int a = 0; a < A; ++a) {
            const int64_t na = tail[a] - head[a];
            if (na == 0) continue;
            double s = 0.0;
            for (int64_t k = head[a]; k < tail[a]; ++k) s += v[q[a][k].id] * exp(-((double)(q[a][k].deadline - T) * 1e-9 / tau));
            const double pr = s / (double)na;
            if (best_a < 0) { best_a = a; best_p = pr; }
            else if (pr > best_p) { second_p = best_p; best_a = a; best_p = pr; }
            else if (pr < best_p && pr > second_p) second_p = pr;
        }
        const int a = best_a, g0 = first_model(p, a / GW), M = p->models_per_app[a / GW];
        const int64_t na = tail[a] - head[a];
        const int pen = p->penalty_kind ? p->penalty_kind[a / GW] : ORC_PEN_STEP;
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
                    u += acc[m->id * MM + j] * (1.0 - orc_penalty(pen, m->deadline, arrival[m->id], e));
                }
                if (best_j < 0) { best_j = j; best_b = (int)b; best_bp = bp; best_e = e; best_u = u; }
                else if (u > best_u) { second_u = best_u; best_j = j; best_b = (int)b; best_bp = bp; best_e = e; best_u = u; }
                else if (u < best_u && u > second_u) second_u = u;
            }
        }
        for (int64_t k = 0; k < best_bp; ++k) {
            orc_req_rec *r = &reqs[q[a][head[a] + k].id];
            r->status = ORC_SCHEDULED; r->round = (int32_t)round; r->model = g0 + best_j; r->worker = wk; r->order = next_order++;
        }
        head[a] += best_bp;
        if (rounds && round < cap) {
            orc_round_rec *rr = &rounds[round];
            rr->instance = 0; rr->round = (int32_t)round; rr->app = a / GW; rr->model = g0 + best_j;
            rr->batch = best_b; rr->n_members = (int32_t)best_bp; rr->n_expired = exp_since;
            rr->label = label ? a % GW - 1 : -1; rr->worker = wk; rr->pad_ = 0;
            rr->t_start_ns = T; rr->t_end_ns = best_e; rr->utility = best_u; rr->group_priority = best_p;
            rr->util_margin = (second_u == -INFINITY || !(best_u > 0.0)) ? INFINITY : (best_u - second_u) / best_u;
            rr->prio_margin = (second_p == -INFINITY || !(best_p > 0.0)) ? INFINITY : (best_p - second_p) / best_p;
        }
        exp_since = 0;
        t_end[wk] = best_e; loaded_end[wk] = g0 + best_j; ++round;
    }
    *n_rounds = round;
    for (int a = 0; a < A; ++a) free(q[a]);
    free(q); free(head); free(tail); free(arr);
#undef GROUP_OF
    return 0;
}

/* ---------------------------------------------------------------------------------------------
 * SneakPeek model of Section 4.1 as the paper builds it: the evidence y is the vote of the k nearest labelled
 * training points of the request's application (the paper uses an approximate index; here the neighbours are exact:
 * squared Euclidean distance summed feature by feature, ties to the lower reference index), theta is the mean of the
 * Dirichlet posterior of Eq. 10-11, theta_c = (alpha_c + y_c) / (sum alpha + k'), k' = min(k, reference points of the
 * application); without a prior theta = y / k'.  Then Eq. 9, Eq. 12's variance factor and the Section 4.3 label as in
 * score_one.  ref [R][D] in the profiles' feature type, ref_label [R] in 0..C-1, ref_app [R]; instance 0's recall.
 * An application without reference points gets theta = prior mean (or uniform without a prior).
 * ------------------------------------------------------------------------------------------- */
int orc_score_knn(const orc_profiles *p, int k, int64_t R, const void *ref, const int32_t *ref_label, const int32_t *ref_app,
                  int64_t n, const void *feats, const int32_t *app, double *acc_out, double *v_out, double *theta_out,
                  int32_t *label_out)
{
    if (!p || k < 1 || R < 0 || n < 0 || !acc_out || !v_out) return -1;
    const int C = p->n_classes, D = p->feat_dim, MM = max_models(p), SM = sum_models(p);
    (void)SM;
    int bad = 0;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        const int a = app[i];
        if (a < 0 || a >= p->n_apps) { bad = 1; continue; }
        double *bd = (double *)malloc(sizeof(double) * (size_t)k);     /* the k best distances so far, ascending */
        int64_t *bi = (int64_t *)malloc(sizeof(int64_t) * (size_t)k);
        double *theta = (double *)calloc((size_t)C, sizeof(double));
        int found = 0;
        for (int64_t r = 0; r < R; ++r) {
            if (ref_app[r] != a) continue;
            double dist = 0.0;
            for (int d = 0; d < D; ++d) {
                const double diff = widen(feats, p->feat_dtype, i * D + d) - widen(ref, p->feat_dtype, r * D + d);
                dist += diff * diff;
            }
            int pos = found < k ? found : k;                           /* insertion; equal distances keep the earlier index first */
            while (pos > 0 && bd[pos - 1] > dist) --pos;
            if (pos < k) {
                for (int t = (found < k ? found : k - 1); t > pos; --t) { bd[t] = bd[t - 1]; bi[t] = bi[t - 1]; }
                bd[pos] = dist; bi[pos] = r;
                if (found < k) ++found;
            }
        }
        for (int t = 0; t < found; ++t) theta[ref_label[bi[t]]] += 1.0;
        const float *al = p->prior_alpha ? p->prior_alpha + (int64_t)a * C : NULL;
        double asum = 0.0;
        if (al) for (int c = 0; c < C; ++c) asum += (double)al[c];
        for (int c = 0; c < C; ++c) {
            if (al) theta[c] = ((double)al[c] + theta[c]) / (asum + (double)found);
            else theta[c] = found > 0 ? theta[c] / (double)found : 1.0 / (double)C;
        }
        if (label_out) { label_out[i] = -1; for (int c = 0; c < C; ++c) if (theta[c] > 0.5) label_out[i] = c; }
        const int M = p->models_per_app[a], g0 = first_model(p, a);
        double *accr = acc_out + i * MM, mean = 0.0;
        for (int j = 0; j < MM; ++j) accr[j] = 0.0;
        for (int j = 0; j < M; ++j) {
            const float *rc = p->recall + (int64_t)(g0 + j) * C;
            double s = 0.0;
            for (int c = 0; c < C; ++c) s += theta[c] * (double)rc[c];
            accr[j] = s; mean += s;
        }
        mean = mean / M;
        double var = 0.0;
        for (int j = 0; j < M; ++j) var += (accr[j] - mean) * (accr[j] - mean);
        v_out[i] = 1.0 + var / M;
        if (theta_out) memcpy(theta_out + i * C, theta, sizeof(double) * (size_t)C);
        free(bd); free(bi); free(theta);
    }
    return bad ? -1 : 0;
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
