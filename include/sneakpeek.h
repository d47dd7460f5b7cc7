/*
 * sneakpeek.h -- C ABI of the B200 scoring-and-selection library.
 *
 * The library runs, on one GPU, the step an inference-serving scheduler repeats every round in
 * SneakPeek (arXiv 2505.06641): it evaluates a SneakPeek model on every pending request to get a
 * per-class posterior (Section 4.1), turns it into data-aware accuracies of every candidate model
 * variant (Eq. 9), and then runs group-level greedy scheduling rounds (Eq. 12-14, Algorithm 1)
 * with (model variant, batch size) candidates scored by the summed utility of Eq. 2.
 *
 * Conventions
 *   - Every function returns an sp_status; nothing throws or aborts across this boundary.
 *     sp_last_error() gives a text for the last non-OK status of a context.
 *   - "HOST" / "DEVICE" in a comment says where a pointer must point.  Device pointers must belong
 *     to the context's device.  Work is enqueued on the context's CUDA stream and is asynchronous
 *     unless stated; sp_check() waits for it and reports errors found on the device.
 *   - Times are int64 nanoseconds on one common clock.  Model ids are GLOBAL ids
 *     g = (number of models of applications 0..a-1) + j for variant j of application a.
 *   - The context owns the device memory it allocates; caller buffers stay the caller's.
 *   - There is no CPU fallback: without a usable CUDA device every call fails with SP_ECUDA.
 */
#ifndef SNEAKPEEK_H_
#define SNEAKPEEK_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct sp_ctx sp_ctx; /* opaque */

typedef enum {
    SP_OK = 0,
    SP_EINVAL = 1, /* bad argument, shape or value (also: bad value found on the device) */
    SP_ENOMEM = 2, /* device or host allocation failed */
    SP_ECUDA = 3,  /* a CUDA call failed */
    SP_ESTATE = 4, /* call made in the wrong order (no profiles, no scored requests, ...) */
    SP_ELIMIT = 5  /* a device-side iteration limit was hit; results are incomplete */
} sp_status;

enum { SP_F32 = 0, SP_BF16 = 1 };                       /* feature / head-weight storage type */
/* Penalty gamma of Eq. 2 (Section 5.1).  STEP: 1 once the deadline is missed.  LINEAR and SIGMOID degrade the utility
 * after the deadline d over the request's relative deadline delta = d - arrival: with x = (completion - d) / delta,
 * gamma = min(max(x, 0), 1) (LINEAR) or 0 for x <= 0, 1 for x >= 1, 1 / (1 + ((1 - x) / x)^3) in between (SIGMOID).
 * gamma is evaluated in fp64.  A pending request at the head of its queue that is hopeless -- the earliest completion
 * any candidate of its application can still reach misses the deadline (STEP) or lies a whole relative deadline or
 * more after it (x >= 1, tested on the integer times) -- is retired as SP_EXPIRED. */
enum { SP_PEN_STEP = 0, SP_PEN_LINEAR = 1, SP_PEN_SIGMOID = 2 };
enum { SP_PENDING = 0, SP_SCHEDULED = 1, SP_EXPIRED = 2 };

/*
 * Profiles registered for the applications (Section 2.2 / 3.2: per-label accuracy, inference
 * latency and model-load latency of every variant) plus the SneakPeek model itself
 * (Definition 4.1.1), here a linear head per application followed by a softmax, and the
 * Dirichlet prior of Eq. 10.  All pointers are HOST pointers; the arrays are copied to the
 * device during sp_load_profiles() and may be freed afterwards.
 * With n_instances = I > 1 the context holds I independent schedulers that share the shapes
 * below but have their own heads, profiles, clock and queues; every per-instance array then
 * has a leading [I] axis.
 */
typedef struct {
    int32_t n_instances;           /* I >= 1 */
    int32_t n_apps;                /* A >= 1 applications (= request groups of Section 4.2) */
    int32_t n_classes;             /* C >= 1 labels; an application with fewer labels pads with bias -inf, recall 0 */
    int32_t feat_dim;              /* D >= 1 */
    int32_t feat_dtype;            /* SP_F32 or SP_BF16: type of the features AND of head_w */
    const int32_t *models_per_app; /* [A], each >= 1 (shared by all instances) */
    const void *head_w;            /* [I][A][D][C], C fastest */
    const float *head_b;           /* [I][A][C] */
    const float *prior_alpha;      /* [I][A][C] Dirichlet hyper-parameters (Eq. 10), or NULL: theta = softmax output */
    float evidence_k;              /* kappa > 0: the head's output p counts as evidence y = kappa * p in Eq. 11 */
    const float *recall;           /* [I][sumM][C] per-model per-label accuracy in [0,1] */
    const int64_t *lat_alpha_ns;   /* [I][sumM]  batch latency l(m,b) = alpha_m + beta_m * b, both >= 0 */
    const int64_t *lat_beta_ns;    /* [I][sumM] */
    const int64_t *swap_ns;        /* [I][sumM]  time to load model m when another model is resident, >= 0 */
    const int32_t *batch_sizes;    /* [n_batch_sizes] strictly ascending, >= 1 (shared) */
    int32_t n_batch_sizes;         /* 1..16 */
    const int32_t *penalty_kind;   /* [A] SP_PEN_* per application (shared by all instances), or NULL = all step */
    double prio_time_scale_s;      /* tau > 0 in exp(-(d - T)/tau) of Eq. 12, seconds */
} sp_profiles;

/* One executed batch (one greedy pick of Algorithm 1's loop). */
typedef struct {
    int32_t instance, round, app, model, batch, n_members, n_expired, exact;
    int64_t t_start_ns, t_end_ns;
    double utility;        /* summed Eq. 2 utility of the members */
    double group_priority; /* Eq. 14 of the chosen application at t_start */
} sp_round_rec;            /* 64 bytes.  batch = chosen allowed batch size, n_members = min(batch, live);
                              n_expired = requests retired since the previous record; exact = bit 0: the
                              application, bit 1: the candidate was decided by the fp64 re-evaluation */

/* Per-request result: the schedule entry s_ij of Section 3.1 (model = j as a global id, order = s_ij). */
typedef struct {
    int32_t status; /* SP_PENDING / SP_SCHEDULED / SP_EXPIRED */
    int32_t round;  /* round that scheduled or retired it, -1 while pending */
    int32_t model;  /* global model id, -1 unless scheduled */
    int32_t worker; /* worker that runs it (sp_schedule_workers), else 0 */
    int64_t order;  /* 1-based execution order inside its instance, 0 unless scheduled */
} sp_req_rec;       /* 24 bytes */

typedef struct {
    int32_t trace_mode;   /* 0: every scored request is pending at once; 1: a request joins when arrival <= clock */
    int32_t timing;       /* 1: bracket the scoring and the scheduling kernel with CUDA events (see sp_stats) */
    double guard_utility; /* relative margin under which candidate utilities are re-evaluated in fp64; 0 = the
                             default (2e-5), so a zero-initialised struct is safe; (0, 1]: that margin */
    double guard_priority;/* same for group priorities (default 2e-6) */
} sp_options;

typedef struct {
    int64_t kernel_launches;   /* kernels this context has launched so far */
    int64_t rounds;            /* rounds executed since the last sp_reset (all instances) */
    int64_t exact_utility;     /* rounds whose candidate was decided in fp64 */
    int64_t exact_priority;    /* rounds whose application was decided in fp64 */
    int64_t exact_rows;        /* request rows re-scored in fp64 */
    /* With sp_options.timing: device time of the scoring kernel / the scheduling kernel alone, summed over the
     * calls since the previous sp_get_stats() (at most 512 calls are kept), and the number of calls summed. */
    int64_t score_calls, sched_calls;
    double score_kernel_ms, sched_kernel_ms;
    /* Scoring kernel the loaded profiles select: 0 = tiled FP32, 1 = small-head FP32, 2 = tensor-core small heads
     * (tcgen05, tf32 split), 3 = tensor-core bf16 GEMM (tcgen05), 4 = tensor-core fp32 GEMM (tcgen05, tf32 split). */
    int32_t score_kernel, pad_;
} sp_stats;

/* Creates a context on CUDA device `device` that enqueues on `cuda_stream` (a cudaStream_t; NULL = the
 * legacy default stream).  *out is NULL on failure. */
sp_status sp_create(sp_ctx **out, int device, void *cuda_stream);
void sp_destroy(sp_ctx *ctx);
const char *sp_last_error(const sp_ctx *ctx);

/* Validates and uploads the profiles (synchronous).  Drops any scored requests.  Clocks start at 0 with no
 * model resident.  SP_EINVAL on a bad shape/value, naming it in sp_last_error(). */
sp_status sp_load_profiles(sp_ctx *ctx, const sp_profiles *profiles);

/* Fills *out (HOST) with the defaults: snapshot mode, no timing, the default guards.  Needs no GPU. */
void sp_default_options(sp_options *out);
/* Replaces the context's options.  Guards must lie in [0, 1]; 0 selects the default. */
sp_status sp_set_options(sp_ctx *ctx, const sp_options *opt);

/* Sets the clock T and the resident model L (global id, -1 = none) of one instance, or of all (instance = -1). */
sp_status sp_set_clock(sp_ctx *ctx, int32_t instance, int64_t t_ns, int32_t loaded_model);
/* Same with per-instance values; t_ns [I], loaded_model [I] are DEVICE pointers. */
sp_status sp_set_clocks(sp_ctx *ctx, const int64_t *t_ns, const int32_t *loaded_model);

/*
 * Scores n requests (Section 4.1 and Eq. 9, Eq. 12's variance factor) and adds them to the context's request table.
 * The first call after sp_reset() / sp_load_profiles() starts a table with ids 0..n-1.  A further call APPENDS: the new
 * requests get the ids that follow (Section 3.2: requests are enqueued while the scheduler runs), earlier results and
 * the scheduler's state stay, and the next sp_schedule_round() sees the new requests (snapshot mode: at once; trace
 * mode: from their arrival time on, which must not precede the arrival of the last request already in the table).
 * Appending is for single-instance contexts (n_instances == 1; otherwise SP_ESTATE), at most 4,096 calls per table.
 * All pointers are DEVICE pointers and are BORROWED until sp_reset(), sp_load_profiles() or sp_destroy(): the
 * scheduler reads deadlines and, for near-ties, the raw features again.  (From the first append on the context keeps
 * its own copy of app / arrival_ns / deadline_ns, 20 bytes per request; the feature matrices stay the caller's.)
 *   feats       [n][D] row-major, float or bf16 as in the profiles; 16-byte aligned
 *   app         [n] application of each request, 0..A-1
 *   arrival_ns  [n]; deadline_ns [n]
 *   instance    [n] instance of each request, non-decreasing; NULL when I == 1.  In trace mode arrivals
 *               must be non-decreasing inside an instance.
 *   acc_out     [n][Mmax] float, optional (NULL): receives the data-aware accuracies of THESE n requests, columns
 *               >= M_app are 0.
 * Violations found on the device (bad app/instance, order) surface as SP_EINVAL from sp_check(); the table is then
 * unusable until sp_reset().
 */
sp_status sp_score(sp_ctx *ctx, int64_t n, const void *feats, const int32_t *app, const int64_t *arrival_ns,
                   const int64_t *deadline_ns, const int32_t *instance, float *acc_out);

/*
 * The SneakPeek model as the paper builds it (Section 4.1): the evidence of a request is the vote of its k nearest
 * labelled reference points among those of its application (exact neighbours: squared Euclidean distance in fp64, ties
 * to the lower index), theta the mean of the Dirichlet posterior of Eq. 10-11 over the vote counts,
 * theta_c = (alpha_c + y_c) / (sum alpha + k'), k' = min(k, reference points of the application); without a prior
 * theta = y / k' (uniform when the application has no reference point).  sp_load_evidence copies the reference set (HOST
 * arrays; single-instance contexts; dropped by sp_load_profiles).  sp_score_knn is sp_score() with that model in place
 * of the linear head (head_w / head_b / evidence_k of the profiles are not used); it starts a table and cannot append.
 */
typedef struct {
    int32_t k;                  /* neighbours, 1..1024 */
    int64_t n_ref;              /* R reference points */
    const void *ref_feats;      /* HOST [R][D], float or bf16 as in the profiles */
    const int32_t *ref_label;   /* HOST [R], 0..C-1 */
    const int32_t *ref_app;     /* HOST [R], 0..A-1 */
} sp_knn_evidence;
sp_status sp_load_evidence(sp_ctx *ctx, const sp_knn_evidence *evidence);
sp_status sp_score_knn(sp_ctx *ctx, int64_t n, const void *feats, const int32_t *app, const int64_t *arrival_ns,
                       const int64_t *deadline_ns, float *acc_out);

/* Copies scores of requests first..first+n-1 to DEVICE buffers: acc [n][Mmax] float and/or v [n] float
 * (v = 1 + population variance of the request's accuracies); either may be NULL. */
sp_status sp_get_scores(sp_ctx *ctx, int64_t first, int64_t n, float *acc, float *v);

/*
 * Runs up to max_rounds greedy rounds per instance back to back on the device (Algorithm 1's loop, one
 * batch per round): arrivals join, hopeless requests are retired, the application with the highest
 * Eq. 14 priority is chosen, every (model, batch size) candidate of it is scored by summed Eq. 2 utility,
 * the best is emitted (ties: lowest application, lowest model, smallest batch), its members leave the
 * queue, the clock advances by the batch latency (+ swap) and the model becomes resident.  An instance
 * stops early when nothing is pending and no arrival is left.
 *   rounds_out  DEVICE [I][cap] or NULL: record k of this call of instance i goes to rounds_out[i*cap + k], k < cap
 *   n_done      DEVICE [I] or NULL: rounds executed by this call
 */
sp_status sp_schedule_round(sp_ctx *ctx, int32_t max_rounds, sp_round_rec *rounds_out, int64_t cap,
                            int32_t *n_done);

/*
 * More ways to schedule a freshly scored SNAPSHOT table (no round run on it yet, not trace mode; otherwise
 * SP_ESTATE).  They first compute the fp64 scores and the data-aware label of every request in one pass over the
 * whole table and take every decision on those, run the table to completion in one call, and write records like
 * sp_schedule_round() (rounds_out DEVICE [I][cap] or NULL, n_done DEVICE [I] or NULL; sp_round_rec.exact carries the
 * sub-group: bits 8 and up hold predicted label + 1, 0 = the application's unsplit remainder or no sub-groups).
 *
 * sp_schedule_split: the greedy rounds of Algorithm 1 over data-aware sub-groups (Section 4.3, "Enhancements for Grouped
 *   Scheduling"): requests of an application whose posterior gives one label more than one half form a group of their
 *   own, the others stay together; Eq. 14, the purge and the (model, batch size) candidates apply per sub-group.  Ties
 *   between groups go to the lowest application, then the unsplit remainder, then the lowest label.
 * sp_schedule_exhaustive: Algorithm 1's branch for few groups (Section 4.2): every order of the non-empty groups
 *   (applications, or sub-groups when split != 0) times every model per group; a group is served whole on its model,
 *   members in (deadline, id) order in batches of the largest allowed size, nothing is retired; the best total utility
 *   wins (ties: first in lexicographic order of the group order, then of the model choices).  Single-instance contexts;
 *   at most 8 non-empty groups and 2^31 solutions (SP_EINVAL beyond).  Synchronous.  total_out / n_solutions_out: HOST,
 *   optional.
 * sp_schedule_baseline: the request-level baselines of Section 5.1, one request at a time in EDF or Eq. 12 priority
 *   order: SP_BASE_MAXACC_EDF (most accurate model that meets the deadline, else the most accurate of all),
 *   SP_BASE_LO_EDF and SP_BASE_LO_PRIORITY (Eq. 13: highest utility at the time the request starts).  Nothing is retired.
 * sp_get_labels: the labels (-1 = none above one half) to a DEVICE buffer, after one of these calls.
 * sp_set_workers / sp_schedule_workers / sp_get_workers: several workers (Section 6: every model variant has a latency
 *   profile per worker and the schedule gains a worker index).  sp_set_workers registers 1..64 workers with HOST arrays
 *   [W][sumM] (copied; single-instance contexts; dropped by sp_load_profiles).  sp_schedule_workers runs the greedy
 *   rounds (over applications, or sub-groups when split != 0) as list scheduling: every worker starts at the instance's
 *   clock with its resident model; the worker that is free first (lowest clock, then lowest index) takes the next batch,
 *   chosen as in a single-worker round from that worker's profile; a request is retired when no worker could complete
 *   it in time.  sp_req_rec.worker and bits 2..7 of sp_round_rec.exact give the worker.  sp_get_workers copies the
 *   workers' final clocks and resident models to DEVICE buffers t_ns [W], loaded [W]; the instance's clock becomes the
 *   last completion.
 */
enum { SP_BASE_MAXACC_EDF = 0, SP_BASE_LO_EDF = 1, SP_BASE_LO_PRIORITY = 2 };
sp_status sp_set_workers(sp_ctx *ctx, int32_t n_workers, const int64_t *lat_alpha_ns, const int64_t *lat_beta_ns,
                         const int64_t *swap_ns);
sp_status sp_schedule_workers(sp_ctx *ctx, int32_t split, sp_round_rec *rounds_out, int64_t cap, int32_t *n_done);
sp_status sp_get_workers(sp_ctx *ctx, int64_t *t_ns, int32_t *loaded);
sp_status sp_schedule_split(sp_ctx *ctx, sp_round_rec *rounds_out, int64_t cap, int32_t *n_done);
sp_status sp_schedule_exhaustive(sp_ctx *ctx, int32_t split, sp_round_rec *rounds_out, int64_t cap, int32_t *n_done,
                                 double *total_out, int64_t *n_solutions_out);
sp_status sp_schedule_baseline(sp_ctx *ctx, int32_t policy, sp_round_rec *rounds_out, int64_t cap, int32_t *n_done);
sp_status sp_get_labels(sp_ctx *ctx, int64_t first, int64_t n, int32_t *labels);

/* Copies the records of requests first..first+n-1 to a DEVICE buffer. */
sp_status sp_get_requests(sp_ctx *ctx, int64_t first, int64_t n, sp_req_rec *out);
/* Copies every instance's clock and resident model to DEVICE buffers t_ns [I], loaded_model [I]. */
sp_status sp_get_clocks(sp_ctx *ctx, int64_t *t_ns, int32_t *loaded_model);

/* Forgets the scored requests and queues; profiles, options, clocks and resident models stay. */
sp_status sp_reset(sp_ctx *ctx);

/* Waits for the context's stream and returns the first error recorded on the device since the last
 * sp_check(): SP_EINVAL (bad request data), SP_ELIMIT (iteration limit), else SP_OK. */
sp_status sp_check(sp_ctx *ctx);
sp_status sp_get_stats(sp_ctx *ctx, sp_stats *out /* HOST */);

/*
 * Whole path from HOST buffers: uploads the requests, scores them, runs every instance to completion
 * (at most max_rounds rounds each), downloads the results, and waits.  Replaces the request table.
 * feats/app/arrival_ns/deadline_ns/instance as in sp_score() but HOST pointers (pinned memory makes the
 * copies faster); t0_ns [I] and loaded0 [I] (NULL = keep) are the starting clocks and resident models.
 * Outputs, all HOST and optional: reqs_out [n], rounds_out [I][cap], n_done [I].
 */
sp_status sp_run_host(sp_ctx *ctx, int64_t n, const void *feats, const int32_t *app, const int64_t *arrival_ns,
                      const int64_t *deadline_ns, const int32_t *instance, const int64_t *t0_ns,
                      const int32_t *loaded0, int32_t max_rounds, sp_req_rec *reqs_out,
                      sp_round_rec *rounds_out, int64_t cap, int32_t *n_done);

/*
 * Scoring for callers that must not allocate.  (The paper has no counterpart to this entry point; it exists
 * for deployment reasons only.)  Some hosts of this library run with a fixed device-memory budget handed out
 * at start-up -- a serving process that has given all remaining memory to its own pool, or a real-time loop
 * in which a driver allocation (which may block or fail) is not acceptable -- so the context-based calls
 * above, which grow their buffers with cudaMalloc, are closed to them.  This call does steps a1-a4 of
 * sp_score() for ONE instance (no Dirichlet prior) and requests no device memory, neither through CUDA nor
 * through any library: its scratch (per-application counters, prefix sums, the request permutation; about
 * 0.5 MB) is a fixed array inside the library image, which every GPU that loads the library holds until the
 * process ends.  That claim is about the second and later calls on a device.  The FIRST call on a device makes
 * the device current, which creates its primary context and loads the library's module (the 0.5 MB array
 * included) if nothing has done so yet: those are driver allocations, so make that first call at start-up,
 * before the memory budget is handed out.  Like the context-based calls, every call leaves `device` the calling
 * thread's current device.  Error texts are formatted on the host heap.
 *
 *   head      HOST struct; models_per_app is a HOST array, head_w [A][D][C], head_b [A][C], recall [sumM][C]
 *             are DEVICE arrays (inputs, the caller's).
 *   n         0 .. 65,536 requests; larger n is rejected with SP_EINVAL and a message (the array is not grown).
 *   feats     DEVICE [n][D]; app DEVICE [n]; acc_out DEVICE [n][Mmax] float; v_out DEVICE [n] float (outputs).
 *   errbuf    HOST, optional: receives a text when the result is not SP_OK.
 *
 * The call returns when the work is done (it waits for the stream) and reports bad application ids as
 * SP_EINVAL.  The first call on a device looks up the array's device address (once per device); make that
 * first call before starting any stream capture.  All calls in a process share the one array per device: it
 * keeps the last call's contents, the call clears what has to start at zero, and two calls that overlap on
 * the same GPU (different streams or threads) race on it -- serialise them.
 */
typedef struct {
    int32_t n_apps, n_classes, feat_dim, feat_dtype;
    const int32_t *models_per_app; /* HOST [A] */
    const void *head_w;            /* DEVICE [A][D][C] */
    const float *head_b;           /* DEVICE [A][C] */
    const float *recall;           /* DEVICE [sumM][C] */
} sp_static_head;

sp_status sp_score_static(int device, void *cuda_stream, const sp_static_head *head, int64_t n, const void *feats,
                          const int32_t *app, float *acc_out, float *v_out, char *errbuf, int32_t errbuf_len);

#ifdef __cplusplus
}
#endif
#endif /* SNEAKPEEK_H_ */
