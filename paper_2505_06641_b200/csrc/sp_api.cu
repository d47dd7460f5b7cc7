// C ABI of the scoring-and-selection library: context, validation, device buffers, kernel launches.
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "sp_common.cuh"
#include "sp_group.cuh"
#include "sp_score_small.cuh"
#include "sp_score_tiled.cuh"
#include "sp_score_mma.cuh"
#include "sp_score_gemm.cuh"
#include "sp_sched.cuh"
#include "sp_sched_warp.cuh"
#include "sp_presort.cuh"
#include "sp_policies.cuh"
#include "sp_knn.cuh"

using namespace sp;

namespace {

constexpr double kDefaultGuardUtility = 2e-5, kDefaultGuardPriority = 2e-6;
constexpr int64_t kDeferMinRows = 4096;   // single instances above this size get the grid-wide fp64 pass queued behind k_sched
constexpr int kDeferExactRows = 512;      // rows a block re-scores by itself before it asks for that pass
constexpr size_t kMaxSegments = 4096;   // sp_score calls that may build one request table

struct Buf {                     // a device allocation that only grows
    void *p = nullptr;
    size_t bytes = 0;
};

struct HostProfiles {            // host copies of the shared (small) profile arrays
    std::vector<int32_t> models_per_app, batch_sizes;
};

}  // namespace

struct sp_ctx {
    int device = 0;
    cudaStream_t stream = nullptr;
    std::string err;
    bool have_profiles = false;
    bool have_table = false;
    bool sched_started = false;  // a scheduling call has run on the current request table
    HostProfiles hp;
    DevProfiles P{};
    DevTable tb{};
    sp_options opt{0, 0, kDefaultGuardUtility, kDefaultGuardPriority};
    std::vector<cudaEvent_t> ev_score, ev_sched;   // start/stop pairs recorded since the last sp_get_stats
    int64_t launches = 0;
    int sched_threads = 1024;
    int small_ct = 0;            // labels per lane of the small-head kernel, 0 = use the tiled kernel
    size_t small_smem = 0;
    int mma_ct = 0;              // logit columns per epilogue thread of the tensor-core kernel, 0 = not used
    bool gemm_on = false;      // a GEMM-shaped tensor-core kernel scores this context's requests (either flavour)
    bool gemm_f32 = false;       // ... the fp32 (tf32 split) flavour
    int gemm_cp = 0;             // labels per head in the transposed image
    CUtensorMap wt_map, r_map, b_map;
    int n_sms = 1;
    // profile buffers
    Buf W, bias, recall, prior, prior_dot, prior_sum, lat_alpha, lat_beta, swap;
    // per-instance state and scratch
    Buf state, zbuf, flags, stats, cnt, gstart, cursor, small_start, tiled_start, small_tiles, scan_partial, wt_image, gemm_tiles, gemm_counter, gemm_partial, gemm_count;
    // per-request buffers
    Buf acc32, v32, acc64, v64, exact, recs, perm, q_id0, q_id1, q_dl0, q_dl1, q_pw0, q_pw1, sort_scratch;
    // requests appended to a scored table: the context's own copies of application / arrival / deadline, the list of
    // the calls' feature matrices, grouping scratch of an append, temporaries of the queue relocation
    bool own_requests = false;
    std::vector<FeatSeg> segs;
    std::vector<Buf> seg_copies;
    Buf t_app, t_arrival, t_deadline, a_cnt, a_cursor, a_gstart, r_id, r_dl, r_pw;
    // policies decided on fp64 scores: labels, group tables, exhaustive search
    Buf labels, g_key, g_start, g_head, g_count, exh_info, exh_total, exh_sol;
    // k-nearest-neighbour evidence (sp_load_evidence): reference set feature-major in fp64, grouped by application
    int knn_k = 0;
    int64_t knn_R = 0, knn_max_per_app = 0;
    Buf knn_refT, knn_label, knn_start, knn_prior_total, knn_dist;
    int n_workers = 0;           // workers registered with sp_set_workers (0 = none)
    Buf w_alpha, w_beta, w_swap, w_T, w_L;
    bool have_exact_all = false;
    // staging of sp_run_host
    Buf h_feats, h_app, h_arrival, h_deadline, h_instance, h_t0, h_loaded, h_rounds, h_ndone;
};

namespace {

sp_status fail(sp_ctx *c, sp_status s, const std::string &msg) {
    if (c) c->err = msg;
    return s;
}

#define SP_CUDA(ctx, call)                                                                           \
    do {                                                                                             \
        cudaError_t e_ = (call);                                                                     \
        if (e_ != cudaSuccess)                                                                       \
            return fail(ctx, e_ == cudaErrorMemoryAllocation ? SP_ENOMEM : SP_ECUDA,                 \
                        std::string(#call) + ": " + cudaGetErrorString(e_));                         \
    } while (0)

sp_status ensure(sp_ctx *c, Buf &b, size_t bytes) {
    if (bytes <= b.bytes && b.p) return SP_OK;
    if (bytes == 0) bytes = 16;
    if (b.p) {
        SP_CUDA(c, cudaStreamSynchronize(c->stream));
        SP_CUDA(c, cudaFree(b.p));
        b.p = nullptr; b.bytes = 0;
    }
    SP_CUDA(c, cudaMalloc(&b.p, bytes));
    b.bytes = bytes;
    return SP_OK;
}

// Like ensure(), but the first keep_bytes of the old allocation survive; capacity grows geometrically.
sp_status grow(sp_ctx *c, Buf &b, size_t keep_bytes, size_t bytes) {
    if (bytes <= b.bytes && b.p) return SP_OK;
    if (keep_bytes == 0 || !b.p) return ensure(c, b, bytes > 2 * b.bytes ? bytes : 2 * b.bytes);
    const size_t cap = bytes > 2 * b.bytes ? bytes : 2 * b.bytes;
    void *np = nullptr;
    SP_CUDA(c, cudaMalloc(&np, cap));
    cudaError_t e = cudaMemcpyAsync(np, b.p, keep_bytes, cudaMemcpyDeviceToDevice, c->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);
    if (e != cudaSuccess) { cudaFree(np); return fail(c, SP_ECUDA, std::string("grow: ") + cudaGetErrorString(e)); }
    cudaFree(b.p);
    b.p = np; b.bytes = cap;
    return SP_OK;
}

void release(Buf &b) {
    if (b.p) cudaFree(b.p);
    b.p = nullptr; b.bytes = 0;
}

// Forgets the request table (host side): the buffers stay allocated for the next one.
void drop_table(sp_ctx *c);

#define SP_TRY(expr)                       \
    do {                                   \
        sp_status s_ = (expr);             \
        if (s_ != SP_OK) return s_;        \
    } while (0)

void drop_table(sp_ctx *c) {
    c->have_table = false;
    c->sched_started = false;
    c->own_requests = false;
    c->have_exact_all = false;
    c->tb.n = 0;
    c->segs.clear();
    for (Buf &b : c->seg_copies) release(b);     // cudaFree waits for kernels that may still read them
    c->seg_copies.clear();
}

sp_status upload(sp_ctx *c, Buf &b, const void *host, size_t bytes) {
    SP_TRY(ensure(c, b, bytes));
    SP_CUDA(c, cudaMemcpyAsync(b.p, host, bytes, cudaMemcpyHostToDevice, c->stream));
    return SP_OK;
}

sp_status launched(sp_ctx *c, const char *what) {
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(c, SP_ECUDA, std::string(what) + ": " + cudaGetErrorString(e));
    ++c->launches;
    return SP_OK;
}

// mode 0: full reset (clock 0, nothing resident); mode 1: forget queues, keep clock and resident model
__global__ void k_state_reset(InstState *st, int n_inst, int mode) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_inst) return;
    InstState s = st[i];
    if (mode == 0) { s.T = 0; s.L = -1; }
    s.next_order = 1; s.Tref = 0; s.inserted = 0; s.round = 0; s.exp_since = 0; s.started = 0; s.handed = 0; s.pad_ = 0;
    for (int a = 0; a < kMaxApps; ++a) { s.head[a] = 0; s.tail[a] = 0; s.cur[a] = 0; }
    st[i] = s;
}

__global__ void k_set_clock(InstState *st, int n_inst, int only, int64_t t, int32_t loaded) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_inst || (only >= 0 && i != only)) return;
    st[i].T = t; st[i].L = loaded;
}

// per-instance values; a null vector keeps what is there
__global__ void k_set_clocks(InstState *st, int n_inst, const int64_t *tv, const int32_t *lv) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_inst) return;
    if (tv) st[i].T = tv[i];
    if (lv) st[i].L = lv[i];
}

__global__ void k_get_clock(const InstState *st, int n_inst, int64_t *t, int32_t *l) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_inst) return;
    if (t) t[i] = st[i].T;
    if (l) l[i] = st[i].L;
}

constexpr size_t kMaxTimedCalls = 512;

// Records an event on the context's stream and keeps it in `list` (timing option only).
sp_status mark(sp_ctx *c, std::vector<cudaEvent_t> &list) {
    if (!c->opt.timing || list.size() >= 2 * kMaxTimedCalls) return SP_OK;
    cudaEvent_t e;
    SP_CUDA(c, cudaEventCreate(&e));
    list.push_back(e);
    SP_CUDA(c, cudaEventRecord(e, c->stream));
    return SP_OK;
}

double drain_events(std::vector<cudaEvent_t> &list, int64_t *calls) {
    double ms = 0.0;
    *calls = 0;
    for (size_t k = 0; k + 1 < list.size(); k += 2) {
        float t = 0.f;
        if (cudaEventElapsedTime(&t, list[k], list[k + 1]) == cudaSuccess) { ms += t; ++*calls; }
    }
    for (cudaEvent_t e : list) cudaEventDestroy(e);
    list.clear();
    return ms;
}

int small_ct_for(int C) { return C <= 10 ? 5 : C <= 20 ? 10 : C <= 32 ? 16 : C <= 64 ? 32 : 0; }

template <int CT>
sp_status launch_small(sp_ctx *c, const DevTable &tv, int grid, float *acc_out) {
    auto kern = k_score_small<CT>;
    SP_CUDA(c, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)c->small_smem));
    kern<<<grid, kSmallThreads, c->small_smem, c->stream>>>(c->P, tv, (const int4 *)c->small_tiles.p, acc_out);
    return launched(c, "k_score_small");
}

// cuTensorMapEncodeTiled through the runtime's driver entry-point lookup (the library does not link libcuda).
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// Tensor map over the fp32 feature matrix [n][D]: boxes of 128 requests x 32 features, 128-byte swizzle,
// zeros outside the matrix.
sp_status feature_map(sp_ctx *c, CUtensorMap *map, const void *feats, int64_t n, int D) {
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return fail(c, SP_ECUDA, "cuTensorMapEncodeTiled is not available from this driver");
    const cuuint64_t dims[2] = {(cuuint64_t)D, (cuuint64_t)n};
    const cuuint64_t strides[1] = {(cuuint64_t)D * 4};
    const cuuint32_t box[2] = {(cuuint32_t)mma::kSlabK, (cuuint32_t)mma::kRows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void *>(feats), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(c, SP_ECUDA, "cuTensorMapEncodeTiled failed with code " + std::to_string((int)r));
    return SP_OK;
}

// Plain 2-D tensor map over a row-major matrix [rows][cols] of `esz`-byte elements, boxes of box_rows x box_cols.
sp_status matrix_map(sp_ctx *c, CUtensorMap *map, const void *ptr, CUtensorMapDataType dt, int esz, int64_t rows, int64_t cols,
                     int box_rows, int box_cols, CUtensorMapSwizzle swz) {
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return fail(c, SP_ECUDA, "cuTensorMapEncodeTiled is not available from this driver");
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)cols * esz};
    const cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = enc(map, dt, 2, const_cast<void *>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(c, SP_ECUDA, "cuTensorMapEncodeTiled failed with code " + std::to_string((int)r));
    return SP_OK;
}

template <int CT, bool PRIOR>
sp_status launch_mma_p(sp_ctx *c, const CUtensorMap &map, const mma::Params &prm) {
    auto kern = mma::k_score_mma<CT, PRIOR>;
    SP_CUDA(c, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, mma::Smem::bytes));
    const int grid = prm.n_tiles < c->n_sms ? prm.n_tiles : c->n_sms;
    kern<<<grid, mma::kThreads, mma::Smem::bytes, c->stream>>>(map, prm);
    return launched(c, "k_score_mma");
}
template <int CT>
sp_status launch_mma(sp_ctx *c, const CUtensorMap &map, const mma::Params &prm) {
    return prm.P.prior ? launch_mma_p<CT, true>(c, map, prm) : launch_mma_p<CT, false>(c, map, prm);
}


// Launches the scoring kernel the loaded profiles select over the rows of `tv` (a table of its own: rows 0..tv.n-1,
// grouping counts and prefix already in tv.cnt / tv.gstart).
sp_status score_rows(sp_ctx *c, const DevTable &tv, float *acc_out) {
    const DevProfiles &P = c->P;
    const int64_t n = tv.n;
    const size_t nkeys = (size_t)P.I * P.A;
    const unsigned gb = (unsigned)((n + 255) / 256);
    int grid = 0;
    if (c->small_ct || c->mma_ct) {
        if (n / kSmallRows + P.I > 0x7fffffff / 2) return fail(c, SP_EINVAL, "too many requests for one call");
        grid = (int)(n / kSmallRows + P.I);
        SP_TRY(ensure(c, c->small_tiles, (size_t)grid * sizeof(int4)));
        k_small_tiles<<<(grid + 255) / 256, 256, 0, c->stream>>>(P, tv, (const int32_t *)c->small_start.p, grid,
                                                                 (int4 *)c->small_tiles.p, (const int *)c->flags.p);
        SP_TRY(launched(c, "k_small_tiles"));
    }
    int n_tiles = 0;
    if (c->gemm_on) {
        k_group_scatter<<<gb, 256, 0, c->stream>>>(P, tv, (const int *)c->flags.p);
        SP_TRY(launched(c, "k_group_scatter"));
        if (n / gemm::kGRows + (int64_t)nkeys > 0x3fffffff) return fail(c, SP_EINVAL, "too many requests for one call");
        n_tiles = (int)(n / gemm::kGRows + (int64_t)nkeys);
        SP_TRY(ensure(c, c->gemm_tiles, (size_t)n_tiles * sizeof(int4)));
        SP_TRY(ensure(c, c->gemm_counter, 16));
        SP_CUDA(c, cudaMemsetAsync(c->gemm_tiles.p, 0xFF, (size_t)n_tiles * sizeof(int4), c->stream));
        SP_CUDA(c, cudaMemsetAsync(c->gemm_counter.p, 0, 16, c->stream));
        gemm::k_gemm_tiles<<<(unsigned)((nkeys + 255) / 256), 256, 0, c->stream>>>((int)nkeys, tv.cnt, tv.gstart, (int4 *)c->gemm_tiles.p,
                                                                                (int *)c->gemm_counter.p, (const int *)c->flags.p);
        SP_TRY(launched(c, "k_gemm_tiles"));
    }
    CUtensorMap x_map;
    if (c->mma_ct) SP_TRY(feature_map(c, &x_map, tv.feats, n, P.D));
    SP_TRY(mark(c, c->ev_score));
    if (c->mma_ct) {
        mma::Params prm{P, tv, (const int4 *)c->small_tiles.p, grid, acc_out, (int *)c->flags.p};
        switch (c->mma_ct) {
            case 8: SP_TRY(launch_mma<8>(c, x_map, prm)); break;
            case 16: SP_TRY(launch_mma<16>(c, x_map, prm)); break;
            case 24: SP_TRY(launch_mma<24>(c, x_map, prm)); break;
            case 32: SP_TRY(launch_mma<32>(c, x_map, prm)); break;
            case 48: SP_TRY(launch_mma<48>(c, x_map, prm)); break;
            default: SP_TRY(launch_mma<64>(c, x_map, prm)); break;
        }
    } else if (c->small_ct) {
        switch (c->small_ct) {
            case 5: SP_TRY(launch_small<5>(c, tv, grid, acc_out)); break;
            case 10: SP_TRY(launch_small<10>(c, tv, grid, acc_out)); break;
            case 16: SP_TRY(launch_small<16>(c, tv, grid, acc_out)); break;
            default: SP_TRY(launch_small<32>(c, tv, grid, acc_out)); break;
        }
    } else if (c->gemm_on) {
        gemm::GParams gp{P, tv, (const int4 *)c->gemm_tiles.p, n_tiles, c->gemm_cp, P.I * P.A * c->gemm_cp, acc_out, (int *)c->flags.p,
                         1, nullptr, nullptr};
        // few tiles per block and at least two label chunks: halves of tiles as work items (see GParams::split)
        const int nc = c->gemm_f32 ? gemm::GCfg<true>::NC : gemm::GCfg<false>::NC;
        if ((P.C + nc - 1) / nc >= 2 && n_tiles < 8 * c->n_sms) {
            SP_TRY(ensure(c, c->gemm_partial, (size_t)n_tiles * 2 * gemm::kMergeFloats * gemm::kGRows * 4));
            SP_TRY(ensure(c, c->gemm_count, (size_t)n_tiles * gemm::kGRows * 4));
            SP_CUDA(c, cudaMemsetAsync(c->gemm_count.p, 0, (size_t)n_tiles * gemm::kGRows * 4, c->stream));
            gp.split = 2; gp.partial = (float *)c->gemm_partial.p; gp.part_count = (int *)c->gemm_count.p;
        }
        const int n_items = n_tiles * gp.split;
        const int ggrid = n_items < c->n_sms ? n_items : c->n_sms;
        if (c->gemm_f32) {
            SP_CUDA(c, cudaFuncSetAttribute(gemm::k_score_gemm<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, gemm::GCfg<true>::bytes));
            gemm::k_score_gemm<true><<<ggrid, gemm::GCfg<true>::Threads, gemm::GCfg<true>::bytes, c->stream>>>(c->wt_map, c->r_map, c->b_map, gp);
        } else {
            SP_CUDA(c, cudaFuncSetAttribute(gemm::k_score_gemm<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, gemm::GCfg<false>::bytes));
            gemm::k_score_gemm<false><<<ggrid, gemm::GCfg<false>::Threads, gemm::GCfg<false>::bytes, c->stream>>>(c->wt_map, c->r_map, c->b_map, gp);
        }
        SP_TRY(launched(c, "k_score_gemm"));
    } else {
        k_group_scatter<<<gb, 256, 0, c->stream>>>(P, tv, (const int *)c->flags.p);
        SP_TRY(launched(c, "k_group_scatter"));
        grid = (int)(n / kTiledRows + (int64_t)nkeys);
        if (P.dtype == SP_BF16)
            k_score_tiled<true><<<grid, kTiledThreads, 0, c->stream>>>(P, tv, (const int32_t *)c->tiled_start.p, acc_out,
                                                                    (const int *)c->flags.p);
        else
            k_score_tiled<false><<<grid, kTiledThreads, 0, c->stream>>>(P, tv, (const int32_t *)c->tiled_start.p, acc_out,
                                                                     (const int *)c->flags.p);
        SP_TRY(launched(c, "k_score_tiled"));
    }
    return mark(c, c->ev_score);
}

// k-nearest-neighbour scoring of the rows of `tv` (fresh single-instance table): fp64 throughout, so the rows also get
// their exact scores and labels, and the policies that run on fp64 scores need no second pass.
sp_status score_rows_knn(sp_ctx *c, const DevTable &tv, float *acc_out) {
    const DevProfiles &P = c->P;
    const size_t nn = (size_t)(tv.n > 0 ? tv.n : 1);
    SP_TRY(ensure(c, c->labels, nn * 4));
    int64_t blocks = (tv.n + kKnnWarps - 1) / kKnnWarps;
    if (blocks > (int64_t)c->n_sms * 4) blocks = (int64_t)c->n_sms * 4;
    const int64_t stride = c->knn_max_per_app > 0 ? c->knn_max_per_app : 1;
    SP_TRY(ensure(c, c->knn_dist, (size_t)blocks * kKnnWarps * stride * 8));
    KnnParams kp{};
    kp.P = P; kp.tb = tv; kp.k = c->knn_k; kp.R = c->knn_R;
    kp.refT = (const double *)c->knn_refT.p; kp.ref_label = (const int32_t *)c->knn_label.p;
    kp.app_start = (const int64_t *)c->knn_start.p;
    kp.prior_total = P.prior ? (const double *)c->knn_prior_total.p : nullptr;
    kp.dist = (double *)c->knn_dist.p; kp.dist_stride = stride;
    kp.labels = (int32_t *)c->labels.p; kp.acc_out = acc_out; kp.flags = (const int *)c->flags.p;
    if (P.prior) {                                   // sum of the hyper-parameters per application, label by label in fp64
        std::vector<float> al((size_t)P.A * P.C);
        SP_CUDA(c, cudaMemcpyAsync(al.data(), P.prior, al.size() * 4, cudaMemcpyDeviceToHost, c->stream));
        SP_CUDA(c, cudaStreamSynchronize(c->stream));
        std::vector<double> tot((size_t)P.A, 0.0);
        for (int a = 0; a < P.A; ++a)
            for (int k = 0; k < P.C; ++k) tot[(size_t)a] += (double)al[(size_t)a * P.C + k];
        SP_TRY(upload(c, c->knn_prior_total, tot.data(), tot.size() * 8));
        SP_CUDA(c, cudaStreamSynchronize(c->stream));
        kp.prior_total = (const double *)c->knn_prior_total.p;
    }
    const size_t smem = (size_t)kKnnWarps * (P.D + P.C) * 8;
    SP_CUDA(c, cudaFuncSetAttribute(k_score_knn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    SP_TRY(mark(c, c->ev_score));
    k_score_knn<<<(unsigned)blocks, kKnnWarps * 32, smem, c->stream>>>(kp);
    SP_TRY(launched(c, "k_score_knn"));
    c->have_exact_all = true;
    return mark(c, c->ev_score);
}

// Appending requests changes the size of every application's queue region (regions are laid out back to back, sized by
// the number of requests of the application scored so far).  One block: the live part of every queue is copied out
// (phase 1) and back in at the start of its new region in queue copy 0 (phase 2); heads, tails and region starts follow.
__global__ void __launch_bounds__(1024)
k_queue_regrow(InstState *state, int A, int64_t *qstart, const int32_t *add_cnt, int64_t *q_id0, int64_t *q_id1,
               int64_t *q_dl0, int64_t *q_dl1, double *q_pw0, double *q_pw1, int64_t *t_id, int64_t *t_dl, double *t_pw,
               const int *flags) {
    __shared__ int64_t s_old[kMaxApps + 1], s_new[kMaxApps + 1], s_live[kMaxApps + 1];
    __shared__ int s_head[kMaxApps], s_cur[kMaxApps];
    if (flags[1]) return;                    // the appended rows were rejected: the table is unusable until sp_reset
    const int tid = threadIdx.x, NT = blockDim.x;
    if (tid == 0) {
        s_new[0] = 0; s_live[0] = 0;
        for (int a = 0; a < A; ++a) {
            s_old[a] = qstart[a];
            s_new[a + 1] = s_new[a] + (qstart[a + 1] - qstart[a]) + add_cnt[a];
            s_live[a + 1] = s_live[a] + (state->tail[a] - state->head[a]);
            s_head[a] = state->head[a]; s_cur[a] = state->cur[a];
        }
    }
    __syncthreads();
    const int64_t total = s_live[A];
    for (int64_t f = tid; f < total; f += NT) {
        int a = 0;
        while (f >= s_live[a + 1]) ++a;
        const int64_t src = s_old[a] + s_head[a] + (f - s_live[a]);
        t_id[f] = (s_cur[a] ? q_id1 : q_id0)[src];
        t_dl[f] = (s_cur[a] ? q_dl1 : q_dl0)[src];
        t_pw[f] = (s_cur[a] ? q_pw1 : q_pw0)[src];
    }
    __threadfence_block();
    __syncthreads();
    for (int64_t f = tid; f < total; f += NT) {
        int a = 0;
        while (f >= s_live[a + 1]) ++a;
        const int64_t dst = s_new[a] + (f - s_live[a]);
        q_id0[dst] = t_id[f]; q_dl0[dst] = t_dl[f]; q_pw0[dst] = t_pw[f];
    }
    __syncthreads();
    if (tid == 0) {
        for (int a = 0; a < A; ++a) {
            state->tail[a] = (int32_t)(s_live[a + 1] - s_live[a]); state->head[a] = 0; state->cur[a] = 0;
            qstart[a] = s_new[a];
        }
        qstart[A] = s_new[A];
    }
}

// Sorts the n keys in the context's sort scratch with the whole GPU (bitonic network, see sp_presort.cuh).
sp_status presort_network(sp_ctx *c, int64_t n) {
    SortKey *keys = (SortKey *)c->sort_scratch.p;
    const unsigned nblk = (unsigned)((n + kPresortChunk - 1) / kPresortChunk);
    const size_t psm = (size_t)kPresortChunk * sizeof(SortKey);
    SP_CUDA(c, cudaFuncSetAttribute(k_presort_local, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)psm));
    k_presort_local<<<nblk, kPresortThreads, psm, c->stream>>>(keys, n, 2, kPresortChunk);
    SP_TRY(launched(c, "k_presort_local"));
    int64_t p2 = 1;
    while (p2 < n) p2 <<= 1;
    const int64_t n_pairs = p2 >> 1;
    for (int64_t k = 2 * (int64_t)kPresortChunk; k <= p2; k <<= 1) {
        for (int64_t j = k >> 1; j >= kPresortChunk; j >>= 1) {
            k_presort_global<<<(unsigned)((n_pairs + 255) / 256), 256, 0, c->stream>>>(keys, n, k, j, n_pairs);
            SP_TRY(launched(c, "k_presort_global"));
        }
        k_presort_local<<<nblk, kPresortThreads, psm, c->stream>>>(keys, n, k, k);
        SP_TRY(launched(c, "k_presort_local"));
    }
    return SP_OK;
}

// Common start of the calls that schedule on fp64 scores: the table must be fresh and in snapshot mode; every request
// gets its fp64 scores and label (one grid-wide pass, kept until the table changes); the group tables are sized.
sp_status policy_prologue(sp_ctx *c, const char *who, GroupParams *gp, bool use_labels, sp_round_rec *rounds_out, int64_t cap,
                          int32_t *n_done) {
    if (!c->have_table) return fail(c, SP_ESTATE, "no scored requests");
    if (c->opt.trace_mode) return fail(c, SP_ESTATE, std::string(who) + " works on a snapshot: trace mode is not supported");
    if (c->sched_started) return fail(c, SP_ESTATE, std::string(who) + " needs a table no round has run on yet; call sp_reset and score again");
    if (cap < 0) return fail(c, SP_EINVAL, "cap must be >= 0");
    SP_CUDA(c, cudaSetDevice(c->device));
    const DevProfiles &P = c->P;
    const int64_t n = c->tb.n;
    const size_t nn = (size_t)(n > 0 ? n : 1);
    SP_TRY(ensure(c, c->labels, nn * 4));
    SP_TRY(ensure(c, c->g_key, (nn + P.I) * 4));
    SP_TRY(ensure(c, c->g_start, (nn + P.I) * 4));
    SP_TRY(ensure(c, c->g_head, (nn + P.I) * 4));
    SP_TRY(ensure(c, c->g_count, (size_t)P.I * 4));
    if (!c->have_exact_all && n > 0) {
        int warps = 8;
        while (warps > 1 && (size_t)warps * P.C * 8 > 200 * 1024) warps >>= 1;
        const size_t smem = (size_t)warps * P.C * 8;
        SP_CUDA(c, cudaFuncSetAttribute(k_exact_all, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        int64_t blocks = (n + warps - 1) / warps;
        if (blocks > (int64_t)c->n_sms * 8) blocks = (int64_t)c->n_sms * 8;
        k_exact_all<<<(unsigned)blocks, warps * 32, smem, c->stream>>>(P, c->tb, (int32_t *)c->labels.p, (const int *)c->flags.p,
                                                                       nullptr, nullptr);
        SP_TRY(launched(c, "k_exact_all"));
        c->have_exact_all = true;
    }
    *gp = GroupParams{};
    gp->P = P; gp->tb = c->tb; gp->state = (InstState *)c->state.p;
    gp->labels = use_labels ? (const int32_t *)c->labels.p : nullptr;
    gp->q_id = (int64_t *)c->q_id0.p; gp->q_dl = (int64_t *)c->q_dl0.p; gp->q_pw = (double *)c->q_pw0.p;
    gp->keys = (SortKey *)c->sort_scratch.p;
    gp->g_key = (int32_t *)c->g_key.p; gp->g_start = (int32_t *)c->g_start.p; gp->g_head = (int32_t *)c->g_head.p;
    gp->g_count = (int32_t *)c->g_count.p;
    gp->flags = (int *)c->flags.p; gp->stats = (unsigned long long *)c->stats.p;
    gp->rounds_out = rounds_out; gp->cap = rounds_out ? cap : 0; gp->n_done = n_done;
    gp->bmax = P.batch[P.nB - 1];
    const int64_t per_inst = P.I > 1 ? (n + P.I - 1) / P.I * 2 : n;
    int sort_cap = P.I > 1 ? 1024 : 4096;
    while (sort_cap > 64 && sort_cap / 2 >= per_inst) sort_cap /= 2;
    gp->sort_cap = sort_cap;
    gp->presorted = 0;
    c->sched_started = true;
    return SP_OK;
}

}  // namespace

// =================================================================================================
extern "C" {

sp_status sp_create(sp_ctx **out, int device, void *cuda_stream) {
    if (!out) return SP_EINVAL;
    *out = nullptr;
    int n_dev = 0;
    if (cudaGetDeviceCount(&n_dev) != cudaSuccess || device < 0 || device >= n_dev) return SP_ECUDA;
    if (cudaSetDevice(device) != cudaSuccess) return SP_ECUDA;
    sp_ctx *c = new (std::nothrow) sp_ctx();
    if (!c) return SP_ENOMEM;
    c->device = device;
    c->stream = (cudaStream_t)cuda_stream;
    if (cudaDeviceGetAttribute(&c->n_sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || c->n_sms < 1) c->n_sms = 1;
    if (ensure(c, c->flags, 4 * sizeof(int)) != SP_OK || ensure(c, c->stats, 4 * sizeof(unsigned long long)) != SP_OK ||
        cudaMemsetAsync(c->flags.p, 0, 4 * sizeof(int), c->stream) != cudaSuccess ||
        cudaMemsetAsync(c->stats.p, 0, 4 * sizeof(unsigned long long), c->stream) != cudaSuccess) {
        delete c;
        return SP_ECUDA;
    }
    *out = c;
    return SP_OK;
}

void sp_destroy(sp_ctx *c) {
    if (!c) return;
    cudaSetDevice(c->device);
    cudaStreamSynchronize(c->stream);
    int64_t dummy;
    drain_events(c->ev_score, &dummy);
    drain_events(c->ev_sched, &dummy);
    Buf *all[] = {&c->W, &c->bias, &c->recall, &c->prior, &c->prior_dot, &c->prior_sum, &c->lat_alpha, &c->lat_beta,
                  &c->swap, &c->state, &c->zbuf, &c->flags, &c->stats, &c->cnt, &c->gstart, &c->cursor,
                  &c->small_start, &c->tiled_start, &c->small_tiles, &c->scan_partial, &c->wt_image, &c->gemm_tiles, &c->gemm_counter, &c->gemm_partial, &c->gemm_count, &c->acc32, &c->v32, &c->acc64, &c->v64, &c->exact, &c->recs,
                  &c->perm, &c->q_id0, &c->q_id1, &c->q_dl0, &c->q_dl1, &c->q_pw0, &c->q_pw1, &c->sort_scratch,
                  &c->h_feats, &c->h_app, &c->h_arrival, &c->h_deadline, &c->h_instance, &c->h_t0, &c->h_loaded,
                  &c->h_rounds, &c->h_ndone, &c->t_app, &c->t_arrival, &c->t_deadline, &c->a_cnt, &c->a_cursor,
                  &c->a_gstart, &c->r_id, &c->r_dl, &c->r_pw, &c->labels, &c->g_key, &c->g_start, &c->g_head, &c->g_count,
                  &c->exh_info, &c->exh_total, &c->exh_sol, &c->w_alpha, &c->w_beta, &c->w_swap, &c->w_T, &c->w_L,
                  &c->knn_refT, &c->knn_label, &c->knn_start, &c->knn_prior_total, &c->knn_dist};
    for (Buf *b : all) release(*b);
    for (Buf &b : c->seg_copies) release(b);
    delete c;
}

const char *sp_last_error(const sp_ctx *c) { return c ? c->err.c_str() : "null context"; }

sp_status sp_load_profiles(sp_ctx *c, const sp_profiles *p) {
    if (!c) return SP_EINVAL;
    if (!p) return fail(c, SP_EINVAL, "profiles is NULL");
    SP_CUDA(c, cudaSetDevice(c->device));
    const int I = p->n_instances, A = p->n_apps, C = p->n_classes, D = p->feat_dim, nB = p->n_batch_sizes;
    if (I < 1) return fail(c, SP_EINVAL, "n_instances must be >= 1");
    if (A < 1 || A > kMaxApps) return fail(c, SP_EINVAL, "n_apps must be 1..16");
    if (C < 1 || C > kMaxClasses) return fail(c, SP_EINVAL, "n_classes must be 1..4096");
    if (D < 1) return fail(c, SP_EINVAL, "feat_dim must be >= 1");
    if (p->feat_dtype != SP_F32 && p->feat_dtype != SP_BF16) return fail(c, SP_EINVAL, "feat_dtype must be SP_F32 or SP_BF16");
    if (nB < 1 || nB > kMaxBatchSizes) return fail(c, SP_EINVAL, "n_batch_sizes must be 1..16");
    if (!p->models_per_app || !p->head_w || !p->head_b || !p->recall || !p->lat_alpha_ns || !p->lat_beta_ns ||
        !p->swap_ns || !p->batch_sizes)
        return fail(c, SP_EINVAL, "a required profile array is NULL");
    if (!(p->prio_time_scale_s > 0.0) || !std::isfinite(p->prio_time_scale_s))
        return fail(c, SP_EINVAL, "prio_time_scale_s must be positive and finite");
    int sumM = 0, Mmax = 0;
    for (int a = 0; a < A; ++a) {
        const int m = p->models_per_app[a];
        if (m < 1 || m > kMaxModelsPerApp) return fail(c, SP_EINVAL, "models_per_app entries must be 1..16");
        sumM += m; Mmax = m > Mmax ? m : Mmax;
    }
    for (int b = 0; b < nB; ++b) {
        if (p->batch_sizes[b] < 1 || p->batch_sizes[b] > kMaxBatch || (b && p->batch_sizes[b] <= p->batch_sizes[b - 1]))
            return fail(c, SP_EINVAL, "batch_sizes must be strictly ascending in 1..1024");
    }
    if (p->penalty_kind)
        for (int a = 0; a < A; ++a)
            if (p->penalty_kind[a] < SP_PEN_STEP || p->penalty_kind[a] > SP_PEN_SIGMOID)
                return fail(c, SP_EINVAL, "penalty_kind entries must be SP_PEN_STEP, SP_PEN_LINEAR or SP_PEN_SIGMOID");
    const int64_t n_models = (int64_t)I * sumM;
    const int64_t lat_limit = (int64_t)1 << 50;
    for (int64_t k = 0; k < n_models; ++k) {
        const int64_t al = p->lat_alpha_ns[k], be = p->lat_beta_ns[k], sw = p->swap_ns[k];
        if (al < 0 || be < 0 || sw < 0 || al > lat_limit || be > lat_limit / kMaxBatch || sw > lat_limit)
            return fail(c, SP_EINVAL, "latency and swap profiles must be in [0, 2^50] ns");
    }
    for (int64_t k = 0; k < n_models * C; ++k)
        if (!(p->recall[k] >= 0.f && p->recall[k] <= 1.f)) return fail(c, SP_EINVAL, "recall must be in [0,1]");
    if (p->prior_alpha) {
        if (!(p->evidence_k > 0.f)) return fail(c, SP_EINVAL, "evidence_k must be > 0 when a prior is given");
        for (int64_t k = 0; k < (int64_t)I * A * C; ++k)
            if (!(p->prior_alpha[k] >= 0.f) || !std::isfinite(p->prior_alpha[k]))
                return fail(c, SP_EINVAL, "prior_alpha must be finite and >= 0");
    }
    // shared memory the scheduler kernel needs for its candidate tables (sort buffer is sized at launch)
    const int bmax = p->batch_sizes[nB - 1];
    const SchedSmem ss(0, Mmax, bmax, kMaxModelsPerApp * kMaxBatchSizes, sumM, 32);
    if (ss.end > 96 * 1024) return fail(c, SP_EINVAL, "models_per_app x largest batch size is too large for one block");

    c->have_profiles = false;
    c->n_workers = 0;
    c->knn_k = 0;
    drop_table(c);
    c->hp.models_per_app.assign(p->models_per_app, p->models_per_app + A);
    c->hp.batch_sizes.assign(p->batch_sizes, p->batch_sizes + nB);
    const size_t esz = p->feat_dtype == SP_BF16 ? 2 : 4;
    SP_TRY(upload(c, c->W, p->head_w, (size_t)I * A * D * C * esz));
    SP_TRY(upload(c, c->bias, p->head_b, (size_t)I * A * C * 4));
    SP_TRY(upload(c, c->recall, p->recall, (size_t)n_models * C * 4));
    SP_TRY(upload(c, c->lat_alpha, p->lat_alpha_ns, (size_t)n_models * 8));
    SP_TRY(upload(c, c->lat_beta, p->lat_beta_ns, (size_t)n_models * 8));
    SP_TRY(upload(c, c->swap, p->swap_ns, (size_t)n_models * 8));
    std::vector<float> pdot, psum;
    if (p->prior_alpha) {
        // sum_c alpha_c recall[m][c] and sum_c alpha_c: the prior's share of Eq. 9 under the posterior mean
        pdot.resize((size_t)n_models); psum.resize((size_t)I * A);
        for (int i = 0; i < I; ++i) {
            int g = 0;
            for (int a = 0; a < A; ++a) {
                const float *al = p->prior_alpha + ((size_t)i * A + a) * C;
                double s = 0.0;
                for (int k = 0; k < C; ++k) s += (double)al[k];
                psum[(size_t)i * A + a] = (float)s;
                for (int j = 0; j < p->models_per_app[a]; ++j, ++g) {
                    const float *r = p->recall + ((size_t)i * sumM + g) * C;
                    double t = 0.0;
                    for (int k = 0; k < C; ++k) t += (double)al[k] * (double)r[k];
                    pdot[(size_t)i * sumM + g] = (float)t;
                }
            }
        }
        SP_TRY(upload(c, c->prior, p->prior_alpha, (size_t)I * A * C * 4));
        SP_TRY(upload(c, c->prior_dot, pdot.data(), pdot.size() * 4));
        SP_TRY(upload(c, c->prior_sum, psum.data(), psum.size() * 4));
    }
    DevProfiles &P = c->P;
    P = DevProfiles{};
    P.I = I; P.A = A; P.C = C; P.D = D; P.dtype = p->feat_dtype; P.sumM = sumM; P.Mmax = Mmax; P.nB = nB;
    P.W = c->W.p; P.bias = (const float *)c->bias.p; P.recall = (const float *)c->recall.p;
    P.prior = p->prior_alpha ? (const float *)c->prior.p : nullptr;
    P.prior_dot = p->prior_alpha ? (const float *)c->prior_dot.p : nullptr;
    P.prior_sum = p->prior_alpha ? (const float *)c->prior_sum.p : nullptr;
    P.kappa = p->evidence_k;
    P.lat_alpha = (const int64_t *)c->lat_alpha.p; P.lat_beta = (const int64_t *)c->lat_beta.p;
    P.swap = (const int64_t *)c->swap.p;
    P.tau = p->prio_time_scale_s;
    for (int a = 0, g = 0; a <= A; ++a) { P.mfirst[a] = g; if (a < A) g += p->models_per_app[a]; }
    for (int b = 0; b < nB; ++b) P.batch[b] = p->batch_sizes[b];
    for (int a = 0; a < A; ++a) {
        P.pen[a] = p->penalty_kind ? p->penalty_kind[a] : SP_PEN_STEP;
        if (P.pen[a] != SP_PEN_STEP) P.any_soft = 1;
    }

    // kernel choices that depend on the shapes only
    c->sched_threads = I > 1 ? 128 : 1024;
    c->small_ct = 0;
    c->mma_ct = 0;
    c->gemm_on = false;
    c->gemm_f32 = false;
    const bool small_head = p->feat_dtype == SP_F32 && D % 4 == 0 && D <= mma::kMaxD && A * C <= mma::kCols && sumM * ((C + 3) & ~3) <= 1024;
    const bool want_bf16 = p->feat_dtype == SP_BF16 && D % 8 == 0;
    const bool want_f32 = p->feat_dtype == SP_F32 && D % 4 == 0 && !small_head;
    if ((want_bf16 || want_f32) && C % 4 == 0 && C >= 32 && (int64_t)I * A * ((C + 15) & ~15) < (1 << 29) && (int64_t)I * A <= 65535) {
        // GEMM-shaped head: transpose it once into the K-major image the tensor-core kernel streams from
        const int Cp = (C + 15) & ~15;
        const int64_t heads = (int64_t)I * A;
        const dim3 tg((unsigned)((Cp + 31) / 32), (unsigned)((D + 31) / 32), (unsigned)heads);
        if (want_bf16) {
            SP_TRY(ensure(c, c->wt_image, (size_t)heads * Cp * D * 2));
            gemm::k_transpose_head_bf16<<<tg, 256, 0, c->stream>>>((const unsigned short *)c->W.p, (unsigned short *)c->wt_image.p,
                                                                   heads, D, C, Cp);
            SP_TRY(launched(c, "k_transpose_head_bf16"));
            SP_TRY(matrix_map(c, &c->wt_map, c->wt_image.p, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, heads * Cp, D, gemm::GCfg<false>::NC,
                              gemm::GCfg<false>::KSlab, CU_TENSOR_MAP_SWIZZLE_128B));
        } else {
            SP_TRY(ensure(c, c->wt_image, (size_t)2 * heads * Cp * D * 4));
            gemm::k_transpose_head_f32<<<tg, 256, 0, c->stream>>>((const float *)c->W.p, (float *)c->wt_image.p, heads, D, C, Cp);
            SP_TRY(launched(c, "k_transpose_head_f32"));
            SP_TRY(matrix_map(c, &c->wt_map, c->wt_image.p, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, 2 * heads * Cp, D, gemm::GCfg<true>::NC,
                              gemm::GCfg<true>::KSlab, CU_TENSOR_MAP_SWIZZLE_128B));
        }
        const int nc = want_bf16 ? gemm::GCfg<false>::NC : gemm::GCfg<true>::NC;
        SP_TRY(matrix_map(c, &c->r_map, c->recall.p, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, (int64_t)I * sumM, C, kMaxModelsPerApp, nc,
                          CU_TENSOR_MAP_SWIZZLE_NONE));
        SP_TRY(matrix_map(c, &c->b_map, c->bias.p, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, heads, C, 1, nc, CU_TENSOR_MAP_SWIZZLE_NONE));
        c->gemm_on = true;
        c->gemm_f32 = want_f32;
        c->gemm_cp = Cp;
    }
    if (c->gemm_on) {
    } else if (p->feat_dtype == SP_F32 && D % 4 == 0 && D <= mma::kMaxD && A * C <= mma::kCols && sumM * ((C + 3) & ~3) <= 1024) {
        c->mma_ct = C <= 8 ? 8 : C <= 16 ? 16 : C <= 24 ? 24 : C <= 32 ? 32 : C <= 48 ? 48 : 64;
    } else if (p->feat_dtype == SP_F32 && D % 4 == 0 && C <= 64) {
        const int ct = small_ct_for(C);
        const SmallSmem L(A, D, sumM, (ct + 3) & ~3);
        const size_t bytes = (size_t)L.end * sizeof(float);
        if (bytes <= 200 * 1024) { c->small_ct = ct; c->small_smem = bytes; }
    }
    const size_t nkeys = (size_t)I * A;
    SP_TRY(ensure(c, c->state, (size_t)I * sizeof(InstState)));
    SP_TRY(ensure(c, c->zbuf, (size_t)I * (c->sched_threads / 32) * C * sizeof(double)));
    SP_TRY(ensure(c, c->cnt, nkeys * 4));
    SP_TRY(ensure(c, c->cursor, nkeys * 4));
    SP_TRY(ensure(c, c->gstart, (nkeys + 1) * 8));
    SP_TRY(ensure(c, c->tiled_start, (nkeys + 1) * 4));
    SP_TRY(ensure(c, c->small_start, ((size_t)I + 1) * 4));
    SP_CUDA(c, cudaMemsetAsync(c->state.p, 0, (size_t)I * sizeof(InstState), c->stream));
    k_state_reset<<<(I + 255) / 256, 256, 0, c->stream>>>((InstState *)c->state.p, I, 0);
    SP_TRY(launched(c, "k_state_reset"));
    SP_CUDA(c, cudaMemsetAsync(c->flags.p, 0, 2 * sizeof(int), c->stream));
    SP_CUDA(c, cudaStreamSynchronize(c->stream));   // the host arrays may be freed on return
    c->have_profiles = true;
    return SP_OK;
}

void sp_default_options(sp_options *out) {
    if (!out) return;
    out->trace_mode = 0; out->timing = 0;
    out->guard_utility = kDefaultGuardUtility; out->guard_priority = kDefaultGuardPriority;
}

sp_status sp_set_options(sp_ctx *c, const sp_options *o) {
    if (!c) return SP_EINVAL;
    if (!o || !(o->guard_utility >= 0.0) || !(o->guard_priority >= 0.0) || o->guard_utility > 1.0 || o->guard_priority > 1.0)
        return fail(c, SP_EINVAL, "guards must be in [0,1]");
    if (c->have_table && (o->trace_mode != 0) != (c->opt.trace_mode != 0))
        return fail(c, SP_ESTATE, "trace_mode cannot change while requests are scored; call sp_reset first");
    c->opt = *o;
    // a zero-initialised struct asks for the defaults, not for decisions on fp32 sums without a guard band
    if (c->opt.guard_utility == 0.0) c->opt.guard_utility = kDefaultGuardUtility;
    if (c->opt.guard_priority == 0.0) c->opt.guard_priority = kDefaultGuardPriority;
    return SP_OK;
}

sp_status sp_set_clock(sp_ctx *c, int32_t instance, int64_t t_ns, int32_t loaded) {
    if (!c) return SP_EINVAL;
    if (!c->have_profiles) return fail(c, SP_ESTATE, "no profiles loaded");
    if (instance < -1 || instance >= c->P.I || loaded < -1 || loaded >= c->P.sumM)
        return fail(c, SP_EINVAL, "instance or model id out of range");
    SP_CUDA(c, cudaSetDevice(c->device));
    k_set_clock<<<(c->P.I + 255) / 256, 256, 0, c->stream>>>((InstState *)c->state.p, c->P.I, instance, t_ns, loaded);
    return launched(c, "k_set_clock");
}

sp_status sp_set_clocks(sp_ctx *c, const int64_t *t_ns, const int32_t *loaded) {
    if (!c) return SP_EINVAL;
    if (!c->have_profiles) return fail(c, SP_ESTATE, "no profiles loaded");
    SP_CUDA(c, cudaSetDevice(c->device));
    k_set_clocks<<<(c->P.I + 255) / 256, 256, 0, c->stream>>>((InstState *)c->state.p, c->P.I, t_ns, loaded);
    return launched(c, "k_set_clocks");
}

sp_status sp_get_clocks(sp_ctx *c, int64_t *t_ns, int32_t *loaded) {
    if (!c) return SP_EINVAL;
    if (!c->have_profiles) return fail(c, SP_ESTATE, "no profiles loaded");
    SP_CUDA(c, cudaSetDevice(c->device));
    k_get_clock<<<(c->P.I + 255) / 256, 256, 0, c->stream>>>((const InstState *)c->state.p, c->P.I, t_ns, loaded);
    return launched(c, "k_get_clock");
}

sp_status sp_reset(sp_ctx *c) {
    if (!c) return SP_EINVAL;
    if (!c->have_profiles) return fail(c, SP_ESTATE, "no profiles loaded");
    SP_CUDA(c, cudaSetDevice(c->device));
    k_state_reset<<<(c->P.I + 255) / 256, 256, 0, c->stream>>>((InstState *)c->state.p, c->P.I, 1);
    SP_TRY(launched(c, "k_state_reset"));
    SP_CUDA(c, cudaMemsetAsync((int *)c->flags.p + 1, 0, 3 * sizeof(int), c->stream));
    SP_CUDA(c, cudaMemsetAsync(c->stats.p, 0, 4 * sizeof(unsigned long long), c->stream));
    drop_table(c);
    return SP_OK;
}

static sp_status score_impl(sp_ctx *c, int64_t n, const void *feats, const int32_t *app, const int64_t *arrival_ns,
                            const int64_t *deadline_ns, const int32_t *instance, float *acc_out, bool knn) {
    if (!c) return SP_EINVAL;
    if (!c->have_profiles) return fail(c, SP_ESTATE, "no profiles loaded");
    const bool append = c->have_table;
    if (knn && (append || c->knn_k < 1))
        return fail(c, SP_ESTATE, append ? "sp_score_knn starts a table: call sp_reset first" : "no evidence loaded; call sp_load_evidence first");
    if (append && c->P.I != 1)
        return fail(c, SP_ESTATE, "requests can be appended to a single-instance context only; call sp_reset first");
    if (n < 0 || n > ((int64_t)1 << 40)) return fail(c, SP_EINVAL, "n out of range");
    if (n > 0 && (!feats || !app || !arrival_ns || !deadline_ns)) return fail(c, SP_EINVAL, "a request array is NULL");
    if (c->P.I > 1 && n > 0 && !instance) return fail(c, SP_EINVAL, "instance is required when n_instances > 1");
    if (((uintptr_t)feats & 15) != 0) return fail(c, SP_EINVAL, "feats must be 16-byte aligned");
    if (append && n == 0) return SP_OK;
    SP_CUDA(c, cudaSetDevice(c->device));
    const DevProfiles &P = c->P;
    const int64_t n_old = append ? c->tb.n : 0, n_tot = n_old + n;
    if (append && c->segs.size() >= kMaxSegments)
        return fail(c, SP_ESTATE, "too many sp_score calls on one table (4096); call sp_reset and score the pending requests again");
    const size_t nn = (size_t)(n_tot > 0 ? n_tot : 1), nkeys = (size_t)P.I * P.A;
    // per-request buffers of the context: rows 0..n_old-1 are kept when requests are appended
    struct { Buf *b; size_t row_bytes; bool keep; } per_row[] = {
        {&c->acc32, (size_t)P.Mmax * 4, true}, {&c->v32, 4, true}, {&c->acc64, (size_t)P.Mmax * 8, true}, {&c->v64, 8, true},
        {&c->exact, 1, true}, {&c->recs, sizeof(sp_req_rec), true}, {&c->perm, 8, false},
        {&c->q_id0, 8, true}, {&c->q_id1, 8, true}, {&c->q_dl0, 8, true}, {&c->q_dl1, 8, true},
        {&c->q_pw0, 8, true}, {&c->q_pw1, 8, true}, {&c->sort_scratch, sizeof(SortKey), false}};
    for (auto &e : per_row) {
        if (append && e.keep) SP_TRY(grow(c, *e.b, (size_t)n_old * e.row_bytes, nn * e.row_bytes));
        else SP_TRY(ensure(c, *e.b, nn * e.row_bytes));
    }
    DevTable &tb = c->tb;
    if (append) {
        // The scheduler reads application, arrival and deadline by request id, and a table made by several calls has
        // them in several caller arrays: from the first append on the context keeps its own copies (20 bytes per
        // request), and the feature matrices of the calls are found through a segment list.
        const bool migrate = !c->own_requests;
        SP_TRY(grow(c, c->t_app, migrate ? 0 : (size_t)n_old * 4, nn * 4));
        SP_TRY(grow(c, c->t_arrival, migrate ? 0 : (size_t)n_old * 8, nn * 8));
        SP_TRY(grow(c, c->t_deadline, migrate ? 0 : (size_t)n_old * 8, nn * 8));
        if (migrate) {
            if (n_old > 0) {
                SP_CUDA(c, cudaMemcpyAsync(c->t_app.p, tb.app, (size_t)n_old * 4, cudaMemcpyDeviceToDevice, c->stream));
                SP_CUDA(c, cudaMemcpyAsync(c->t_arrival.p, tb.arrival, (size_t)n_old * 8, cudaMemcpyDeviceToDevice, c->stream));
                SP_CUDA(c, cudaMemcpyAsync(c->t_deadline.p, tb.deadline, (size_t)n_old * 8, cudaMemcpyDeviceToDevice, c->stream));
            }
            c->segs.clear();
            c->segs.push_back(FeatSeg{0, tb.feats});
            c->own_requests = true;
        }
        SP_CUDA(c, cudaMemcpyAsync((int32_t *)c->t_app.p + n_old, app, (size_t)n * 4, cudaMemcpyDeviceToDevice, c->stream));
        SP_CUDA(c, cudaMemcpyAsync((int64_t *)c->t_arrival.p + n_old, arrival_ns, (size_t)n * 8, cudaMemcpyDeviceToDevice, c->stream));
        SP_CUDA(c, cudaMemcpyAsync((int64_t *)c->t_deadline.p + n_old, deadline_ns, (size_t)n * 8, cudaMemcpyDeviceToDevice, c->stream));
        c->segs.push_back(FeatSeg{n_old, feats});
        // the list is read by kernels of earlier calls that may still run: a new copy per call, the old ones are
        // released with the table
        Buf seg_dev;
        SP_TRY(ensure(c, seg_dev, c->segs.size() * sizeof(FeatSeg)));
        c->seg_copies.push_back(seg_dev);
        SP_CUDA(c, cudaMemcpyAsync(seg_dev.p, c->segs.data(), c->segs.size() * sizeof(FeatSeg), cudaMemcpyHostToDevice, c->stream));
        SP_CUDA(c, cudaStreamSynchronize(c->stream));      // the host vector may move at the next append
        tb.feats = nullptr; tb.segs = (const FeatSeg *)seg_dev.p; tb.n_segs = (int)c->segs.size();
        tb.app = (const int32_t *)c->t_app.p; tb.arrival = (const int64_t *)c->t_arrival.p;
        tb.deadline = (const int64_t *)c->t_deadline.p;
        SP_TRY(ensure(c, c->a_cnt, nkeys * 4));
        SP_TRY(ensure(c, c->a_cursor, nkeys * 4));
        SP_TRY(ensure(c, c->a_gstart, (nkeys + 1) * 8));
        SP_TRY(ensure(c, c->r_id, nn * 8));
        SP_TRY(ensure(c, c->r_dl, nn * 8));
        SP_TRY(ensure(c, c->r_pw, nn * 8));
    } else {
        tb.feats = feats; tb.segs = nullptr; tb.n_segs = 0; tb.app = app; tb.arrival = arrival_ns; tb.deadline = deadline_ns;
        tb.instance = P.I > 1 ? instance : nullptr;
    }
    tb.n = n_tot;
    tb.acc32 = (float *)c->acc32.p; tb.v32 = (float *)c->v32.p; tb.acc64 = (double *)c->acc64.p;
    tb.v64 = (double *)c->v64.p; tb.exact = (unsigned char *)c->exact.p; tb.recs = (sp_req_rec *)c->recs.p;
    tb.cnt = (int32_t *)c->cnt.p; tb.gstart = (int64_t *)c->gstart.p; tb.perm = (int64_t *)c->perm.p;
    tb.cursor = (int32_t *)c->cursor.p;
    tb.qstart = (const int64_t *)c->gstart.p;

    // The rows this call scores, as a table of their own: results go to rows n_old.. of the context's buffers; the
    // grouping scratch of an append is separate from the queue regions the scheduler works on.
    DevTable tv = tb;
    tv.n = n; tv.feats = feats; tv.segs = nullptr; tv.n_segs = 0; tv.app = app; tv.arrival = arrival_ns; tv.deadline = deadline_ns;
    tv.acc32 = tb.acc32 + n_old * P.Mmax; tv.v32 = tb.v32 + n_old; tv.exact = tb.exact + n_old; tv.recs = tb.recs + n_old;
    if (append) { tv.cnt = (int32_t *)c->a_cnt.p; tv.cursor = (int32_t *)c->a_cursor.p; tv.gstart = (int64_t *)c->a_gstart.p; }

    SP_CUDA(c, cudaMemsetAsync(tv.cnt, 0, nkeys * 4, c->stream));
    SP_CUDA(c, cudaMemsetAsync(tv.cursor, 0, nkeys * 4, c->stream));
    SP_CUDA(c, cudaMemsetAsync((int *)c->flags.p + 2, 0, 2 * sizeof(int), c->stream));   // the new rows have no fp64 scores yet
    const unsigned gb = (unsigned)((n + 255) / 256);
    if (n > 0) {
        k_group_count<<<gb, 256, 0, c->stream>>>(P, tv, c->opt.trace_mode, (int *)c->flags.p,
                                                 append && n_old > 0 ? (const int64_t *)c->t_arrival.p + (n_old - 1) : nullptr);
        SP_TRY(launched(c, "k_group_count"));
    }
    if (nkeys <= 4 * (size_t)kScanChunk) {
        k_group_scan<<<1, 1024, 0, c->stream>>>((int)nkeys, P.A, tv.cnt, tv.gstart, (int32_t *)c->tiled_start.p,
                                                (int32_t *)c->small_start.p);
        SP_TRY(launched(c, "k_group_scan"));
    } else {                                           // many keys: per-block totals, then one scan block per chunk
        const int nblk = (int)(nkeys / kScanChunk + 1);    // covers index nkeys (the grand total) as well
        SP_TRY(ensure(c, c->scan_partial, (size_t)3 * nblk * sizeof(long long)));
        k_group_partials<<<nblk, kScanChunk, 0, c->stream>>>((int)nkeys, P.A, tv.cnt, (long long *)c->scan_partial.p);
        SP_TRY(launched(c, "k_group_partials"));
        k_group_scan_blocks<<<nblk, kScanChunk, 0, c->stream>>>((int)nkeys, P.A, tv.cnt, (const long long *)c->scan_partial.p,
                                                              tv.gstart, (int32_t *)c->tiled_start.p, (int32_t *)c->small_start.p);
        SP_TRY(launched(c, "k_group_scan_blocks"));
    }
    if (n > 0) SP_TRY(knn ? score_rows_knn(c, tv, acc_out) : score_rows(c, tv, acc_out));
    if (append) {
        // make room in every application's queue region for its new requests; live entries move to the new regions
        k_queue_regrow<<<1, 1024, 0, c->stream>>>((InstState *)c->state.p, P.A, (int64_t *)c->gstart.p, (const int32_t *)c->a_cnt.p,
                                                  (int64_t *)c->q_id0.p, (int64_t *)c->q_id1.p, (int64_t *)c->q_dl0.p,
                                                  (int64_t *)c->q_dl1.p, (double *)c->q_pw0.p, (double *)c->q_pw1.p,
                                                  (int64_t *)c->r_id.p, (int64_t *)c->r_dl.p, (double *)c->r_pw.p,
                                                  (const int *)c->flags.p);
        SP_TRY(launched(c, "k_queue_regrow"));
    }
    c->have_table = true;
    if (!append) c->sched_started = false;
    return SP_OK;
}

sp_status sp_score(sp_ctx *c, int64_t n, const void *feats, const int32_t *app, const int64_t *arrival_ns,
                   const int64_t *deadline_ns, const int32_t *instance, float *acc_out) {
    return score_impl(c, n, feats, app, arrival_ns, deadline_ns, instance, acc_out, false);
}

sp_status sp_score_knn(sp_ctx *c, int64_t n, const void *feats, const int32_t *app, const int64_t *arrival_ns,
                       const int64_t *deadline_ns, float *acc_out) {
    return score_impl(c, n, feats, app, arrival_ns, deadline_ns, nullptr, acc_out, true);
}

sp_status sp_load_evidence(sp_ctx *c, const sp_knn_evidence *ev) {
    if (!c) return SP_EINVAL;
    if (!c->have_profiles) return fail(c, SP_ESTATE, "no profiles loaded");
    if (c->P.I != 1) return fail(c, SP_ESTATE, "k-nearest-neighbour evidence is for single-instance contexts");
    if (!ev || ev->k < 1 || ev->k > kKnnMaxK || ev->n_ref < 0 || (ev->n_ref > 0 && (!ev->ref_feats || !ev->ref_label || !ev->ref_app)))
        return fail(c, SP_EINVAL, "bad evidence description (k must be 1..1024, arrays non-NULL)");
    const DevProfiles &P = c->P;
    const int64_t R = ev->n_ref;
    if ((size_t)(P.D + P.C) * 8 * kKnnWarps > 200 * 1024) return fail(c, SP_EINVAL, "feat_dim + n_classes is too large for the neighbour kernel");
    std::vector<int64_t> start((size_t)P.A + 1, 0);
    for (int64_t r = 0; r < R; ++r) {
        if (ev->ref_app[r] < 0 || ev->ref_app[r] >= P.A || ev->ref_label[r] < 0 || ev->ref_label[r] >= P.C)
            return fail(c, SP_EINVAL, "reference point with an application or label out of range");
        ++start[(size_t)ev->ref_app[r] + 1];
    }
    int64_t max_per_app = 0;
    for (int a = 0; a < P.A; ++a) { max_per_app = start[a + 1] > max_per_app ? start[a + 1] : max_per_app; start[a + 1] += start[a]; }
    // stable grouping by application (ties between equal distances go to the lower original index), feature-major, fp64
    std::vector<int64_t> cursor(start.begin(), start.end() - 1);
    std::vector<double> refT((size_t)(R > 0 ? R : 1) * P.D);
    std::vector<int32_t> lab((size_t)(R > 0 ? R : 1));
    for (int64_t r = 0; r < R; ++r) {
        const int64_t pos = cursor[(size_t)ev->ref_app[r]]++;
        lab[(size_t)pos] = ev->ref_label[r];
        for (int d = 0; d < P.D; ++d) {
            double val;
            if (P.dtype == SP_BF16) {
                const uint32_t bits = (uint32_t)((const uint16_t *)ev->ref_feats)[r * P.D + d] << 16;
                float f; std::memcpy(&f, &bits, 4); val = (double)f;
            } else val = (double)((const float *)ev->ref_feats)[r * P.D + d];
            refT[(size_t)d * R + pos] = val;
        }
    }
    SP_CUDA(c, cudaSetDevice(c->device));
    SP_TRY(upload(c, c->knn_refT, refT.data(), refT.size() * 8));
    SP_TRY(upload(c, c->knn_label, lab.data(), lab.size() * 4));
    SP_TRY(upload(c, c->knn_start, start.data(), start.size() * 8));
    SP_CUDA(c, cudaStreamSynchronize(c->stream));      // the host arrays may be freed on return
    c->knn_R = R; c->knn_max_per_app = max_per_app;
    c->knn_k = ev->k;
    return SP_OK;
}

sp_status sp_get_scores(sp_ctx *c, int64_t first, int64_t n, float *acc, float *v) {
    if (!c) return SP_EINVAL;
    if (!c->have_table) return fail(c, SP_ESTATE, "no scored requests");
    if (first < 0 || n < 0 || first + n > c->tb.n) return fail(c, SP_EINVAL, "request range out of bounds");
    SP_CUDA(c, cudaSetDevice(c->device));
    if (acc && n)
        SP_CUDA(c, cudaMemcpyAsync(acc, c->tb.acc32 + first * c->P.Mmax, (size_t)n * c->P.Mmax * 4, cudaMemcpyDeviceToDevice, c->stream));
    if (v && n) SP_CUDA(c, cudaMemcpyAsync(v, c->tb.v32 + first, (size_t)n * 4, cudaMemcpyDeviceToDevice, c->stream));
    return SP_OK;
}

sp_status sp_get_requests(sp_ctx *c, int64_t first, int64_t n, sp_req_rec *out) {
    if (!c) return SP_EINVAL;
    if (!c->have_table) return fail(c, SP_ESTATE, "no scored requests");
    if (first < 0 || n < 0 || first + n > c->tb.n || (n && !out)) return fail(c, SP_EINVAL, "request range out of bounds");
    SP_CUDA(c, cudaSetDevice(c->device));
    if (n) SP_CUDA(c, cudaMemcpyAsync(out, c->tb.recs + first, (size_t)n * sizeof(sp_req_rec), cudaMemcpyDeviceToDevice, c->stream));
    return SP_OK;
}

sp_status sp_schedule_round(sp_ctx *c, int32_t max_rounds, sp_round_rec *rounds_out, int64_t cap, int32_t *n_done) {
    if (!c) return SP_EINVAL;
    if (!c->have_table) return fail(c, SP_ESTATE, "no scored requests");
    if (max_rounds < 0 || cap < 0) return fail(c, SP_EINVAL, "max_rounds and cap must be >= 0");
    SP_CUDA(c, cudaSetDevice(c->device));
    const DevProfiles &P = c->P;
    SchedParams sp{};
    sp.P = P; sp.tb = c->tb; sp.state = (InstState *)c->state.p;
    sp.q_id[0] = (int64_t *)c->q_id0.p; sp.q_id[1] = (int64_t *)c->q_id1.p;
    sp.q_dl[0] = (int64_t *)c->q_dl0.p; sp.q_dl[1] = (int64_t *)c->q_dl1.p;
    sp.q_pw[0] = (double *)c->q_pw0.p; sp.q_pw[1] = (double *)c->q_pw1.p;
    sp.sort_scratch = (SortKey *)c->sort_scratch.p; sp.zbuf = (double *)c->zbuf.p;
    sp.flags = (int *)c->flags.p; sp.stats = (unsigned long long *)c->stats.p;
    sp.trace_mode = c->opt.trace_mode; sp.guard_u = c->opt.guard_utility; sp.guard_p = c->opt.guard_priority;
    sp.max_rounds = max_rounds; sp.rounds_out = rounds_out; sp.cap = rounds_out ? cap : 0; sp.n_done = n_done;
    sp.bmax = P.batch[P.nB - 1];
    // shared-memory sort buffer: whole instance when it fits, else the global scratch takes over
    const int64_t per_inst = P.I > 1 ? (c->tb.n + P.I - 1) / P.I * 2 : c->tb.n;
    int sort_cap = P.I > 1 ? 1024 : 8192;
    while (sort_cap > 64 && sort_cap / 2 >= per_inst) sort_cap /= 2;
    sp.sort_cap = sort_cap;
    // a single instance with a short table is faster with half the threads (cheaper block barriers); the scratch
    // buffers are sized for the full block
    const int nt = P.I == 1 && !c->opt.trace_mode && c->tb.n <= 8192 ? 512 : c->sched_threads;
    sp.zbuf_warps = nt / 32;
    const SchedSmem L(sort_cap, P.Mmax, sp.bmax, kMaxModelsPerApp * kMaxBatchSizes, P.sumM, nt / 32);
    // instantiations: soft penalties or not, at most 4 applications or up to kMaxApps, long queues (one large snapshot)
    const bool longq = P.I == 1 && !c->opt.trace_mode && c->tb.n > 16384;
    void (*sched_kernel)(SchedParams) =
        P.any_soft ? (P.A <= 4 ? k_sched<true, 4, false> : k_sched<true, kMaxApps, false>)
                   : (P.A <= 4 ? (longq ? k_sched<false, 4, true> : k_sched<false, 4, false>)
                               : (longq ? k_sched<false, kMaxApps, true> : k_sched<false, kMaxApps, false>));
    SP_CUDA(c, cudaFuncSetAttribute(sched_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)L.end));
    SP_TRY(mark(c, c->ev_sched));
    // Batched mode, first call on a fresh table: one warp per instance takes every instance that fits its slice of
    // shared memory and, block-wide, the few it has to hand over; no k_sched launch is needed then.
    // (A call for zero rounds changes nothing: it goes to k_sched, which returns before touching any queue.)
    if (P.I > 1 && !c->opt.trace_mode && !c->sched_started && c->tb.n > 0 && max_rounds > 0) {
        int64_t wcap = 32;
        while (wcap < (c->tb.n + P.I - 1) / P.I) wcap <<= 1;
        const WarpSchedSmem W((int)wcap, P.Mmax, sp.bmax, P.any_soft != 0);
        if (wcap <= 2048 && P.sumM <= 32 && W.end * kWarpSchedWarps <= 200 * 1024 && c->sched_threads == kWarpSchedWarps * 32) {
            const int wgrid = (P.I + kWarpSchedWarps - 1) / kWarpSchedWarps;
            // the block-wide scheduler runs inside the same kernel for the instances a warp hands over: its shared
            // memory is laid over the warps' slices
            const size_t wsmem = W.end * kWarpSchedWarps > L.end ? W.end * kWarpSchedWarps : L.end;
            constexpr int kBigCpl = kMaxModelsPerApp * kMaxBatchSizes / 32;
            void (*wk)(SchedParams, int);
            if (P.Mmax <= 8 && P.Mmax * P.nB <= 64 && P.A <= 4)   // short unrolled loops for small model, batch-size and application sets
                wk = P.any_soft ? k_sched_warp<8, 2, true> : k_sched_warp<8, 2, false>;
            else
                wk = P.any_soft ? k_sched_warp<kMaxModelsPerApp, kBigCpl, true> : k_sched_warp<kMaxModelsPerApp, kBigCpl, false>;
            SP_CUDA(c, cudaFuncSetAttribute(wk, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)wsmem));
            wk<<<wgrid, kWarpSchedWarps * 32, wsmem, c->stream>>>(sp, (int)wcap);
            SP_TRY(launched(c, "k_sched_warp"));
            c->sched_started = true;
            return mark(c, c->ev_sched);
        }
    }
    // One large snapshot instance: its keys are sorted by the whole GPU first (k_sched would use one block for it).
    if (P.I == 1 && !c->opt.trace_mode && !c->sched_started && max_rounds > 0 && c->tb.n > sort_cap && c->tb.n < ((int64_t)1 << 31)) {
        k_presort_keys<<<(unsigned)((c->tb.n + 255) / 256), 256, 0, c->stream>>>(c->tb, (SortKey *)c->sort_scratch.p, c->tb.n);
        SP_TRY(launched(c, "k_presort_keys"));
        SP_TRY(presort_network(c, c->tb.n));
        sp.presorted = 1;
    }
    if (max_rounds > 0) c->sched_started = true;
    // One large instance: a near-tie between group priorities may need the fp64 scores of every live request.  Beyond a
    // few hundred rows the block stops before that round; the whole GPU then scores the rows that are not cached yet and
    // a second launch resumes the instance (both return at once when the first launch did not ask for them).
    const bool defer = P.I == 1 && c->tb.n > kDeferMinRows && max_rounds > 0;
    sp.defer_exact_rows = defer ? kDeferExactRows : 0;
    sched_kernel<<<P.I, nt, L.end, c->stream>>>(sp);
    SP_TRY(launched(c, "k_sched"));
    if (defer) {
        int warps = 8;
        while (warps > 1 && (size_t)warps * P.C * 8 > 200 * 1024) warps >>= 1;
        const size_t smem = (size_t)warps * P.C * 8;
        SP_CUDA(c, cudaFuncSetAttribute(k_exact_all, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        int64_t blocks = (c->tb.n + warps - 1) / warps;
        if (blocks > (int64_t)c->n_sms * 8) blocks = (int64_t)c->n_sms * 8;
        k_exact_all<<<(unsigned)blocks, warps * 32, smem, c->stream>>>(P, c->tb, nullptr, (const int *)c->flags.p,
                                                                       (const int *)c->flags.p + 2, (unsigned long long *)c->stats.p);
        SP_TRY(launched(c, "k_exact_all"));
        sp.only_handed = 1; sp.presorted = 0;
        sched_kernel<<<P.I, nt, L.end, c->stream>>>(sp);
        SP_TRY(launched(c, "k_sched"));
    }
    return mark(c, c->ev_sched);
}

sp_status sp_get_labels(sp_ctx *c, int64_t first, int64_t n, int32_t *labels) {
    if (!c) return SP_EINVAL;
    if (!c->have_table || !c->have_exact_all) return fail(c, SP_ESTATE, "labels exist after sp_schedule_split, sp_schedule_exhaustive or sp_schedule_baseline");
    if (first < 0 || n < 0 || first + n > c->tb.n || (n && !labels)) return fail(c, SP_EINVAL, "request range out of bounds");
    SP_CUDA(c, cudaSetDevice(c->device));
    if (n) SP_CUDA(c, cudaMemcpyAsync(labels, (const int32_t *)c->labels.p + first, (size_t)n * 4, cudaMemcpyDeviceToDevice, c->stream));
    return SP_OK;
}

// Greedy rounds over groups (applications or data-aware sub-groups) on the profiles' worker or on the registered workers.
static sp_status run_group_rounds(sp_ctx *c, const char *who, bool use_labels, bool use_workers, sp_round_rec *rounds_out,
                                  int64_t cap, int32_t *n_done) {
    GroupParams gp;
    SP_TRY(policy_prologue(c, who, &gp, use_labels, rounds_out, cap, n_done));
    const DevProfiles &P = c->P;
    if (use_workers) {
        gp.W = c->n_workers;
        gp.w_alpha = (const int64_t *)c->w_alpha.p; gp.w_beta = (const int64_t *)c->w_beta.p; gp.w_swap = (const int64_t *)c->w_swap.p;
        gp.w_T = (int64_t *)c->w_T.p; gp.w_L = (int32_t *)c->w_L.p;
    }
    if (P.I == 1 && c->tb.n > gp.sort_cap && c->tb.n < ((int64_t)1 << 31)) {
        k_group_keys<<<(unsigned)((c->tb.n + 255) / 256), 256, 0, c->stream>>>(gp, c->tb.n);
        SP_TRY(launched(c, "k_group_keys"));
        SP_TRY(presort_network(c, c->tb.n));
        gp.presorted = 1;
    }
    const int nt = P.I > 1 ? 128 : 1024;
    const GroupSchedSmem L(gp.sort_cap, P.Mmax, gp.bmax, P.sumM, nt / 32);
    if (L.end > 220 * 1024) return fail(c, SP_EINVAL, "models_per_app x largest batch size is too large for one block");
    SP_CUDA(c, cudaFuncSetAttribute(k_sched_groups, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)L.end));
    SP_TRY(mark(c, c->ev_sched));
    k_sched_groups<<<P.I, nt, L.end, c->stream>>>(gp);
    SP_TRY(launched(c, "k_sched_groups"));
    return mark(c, c->ev_sched);
}

sp_status sp_schedule_split(sp_ctx *c, sp_round_rec *rounds_out, int64_t cap, int32_t *n_done) {
    if (!c) return SP_EINVAL;
    return run_group_rounds(c, "sp_schedule_split", true, false, rounds_out, cap, n_done);
}

sp_status sp_set_workers(sp_ctx *c, int32_t n_workers, const int64_t *lat_alpha_ns, const int64_t *lat_beta_ns, const int64_t *swap_ns) {
    if (!c) return SP_EINVAL;
    if (!c->have_profiles) return fail(c, SP_ESTATE, "no profiles loaded");
    if (c->P.I != 1) return fail(c, SP_ESTATE, "several workers are for single-instance contexts");
    if (n_workers < 1 || n_workers > kMaxWorkers) return fail(c, SP_EINVAL, "n_workers must be 1..64");
    if (!lat_alpha_ns || !lat_beta_ns || !swap_ns) return fail(c, SP_EINVAL, "a worker profile array is NULL");
    const int64_t nm = (int64_t)n_workers * c->P.sumM, lat_limit = (int64_t)1 << 50;
    for (int64_t k = 0; k < nm; ++k)
        if (lat_alpha_ns[k] < 0 || lat_beta_ns[k] < 0 || swap_ns[k] < 0 || lat_alpha_ns[k] > lat_limit ||
            lat_beta_ns[k] > lat_limit / kMaxBatch || swap_ns[k] > lat_limit)
            return fail(c, SP_EINVAL, "latency and swap profiles must be in [0, 2^50] ns");
    SP_CUDA(c, cudaSetDevice(c->device));
    SP_TRY(upload(c, c->w_alpha, lat_alpha_ns, (size_t)nm * 8));
    SP_TRY(upload(c, c->w_beta, lat_beta_ns, (size_t)nm * 8));
    SP_TRY(upload(c, c->w_swap, swap_ns, (size_t)nm * 8));
    SP_TRY(ensure(c, c->w_T, (size_t)n_workers * 8));
    SP_TRY(ensure(c, c->w_L, (size_t)n_workers * 4));
    SP_CUDA(c, cudaStreamSynchronize(c->stream));     // the host arrays may be freed on return
    c->n_workers = n_workers;
    return SP_OK;
}

sp_status sp_schedule_workers(sp_ctx *c, int32_t split, sp_round_rec *rounds_out, int64_t cap, int32_t *n_done) {
    if (!c) return SP_EINVAL;
    if (c->n_workers < 1) return fail(c, SP_ESTATE, "no workers registered; call sp_set_workers first");
    return run_group_rounds(c, "sp_schedule_workers", split != 0, true, rounds_out, cap, n_done);
}

sp_status sp_get_workers(sp_ctx *c, int64_t *t_ns, int32_t *loaded) {
    if (!c) return SP_EINVAL;
    if (c->n_workers < 1) return fail(c, SP_ESTATE, "no workers registered");
    SP_CUDA(c, cudaSetDevice(c->device));
    if (t_ns) SP_CUDA(c, cudaMemcpyAsync(t_ns, c->w_T.p, (size_t)c->n_workers * 8, cudaMemcpyDeviceToDevice, c->stream));
    if (loaded) SP_CUDA(c, cudaMemcpyAsync(loaded, c->w_L.p, (size_t)c->n_workers * 4, cudaMemcpyDeviceToDevice, c->stream));
    return SP_OK;
}

sp_status sp_schedule_exhaustive(sp_ctx *c, int32_t split, sp_round_rec *rounds_out, int64_t cap, int32_t *n_done,
                                 double *total_out, int64_t *n_solutions_out) {
    if (!c) return SP_EINVAL;
    if (c->have_profiles && c->P.I != 1) return fail(c, SP_ESTATE, "the exhaustive branch is for single-instance contexts");
    GroupParams gp;
    SP_TRY(policy_prologue(c, "sp_schedule_exhaustive", &gp, split != 0, rounds_out, cap, n_done));
    SP_TRY(ensure(c, c->exh_info, sizeof(ExhInfo)));
    ExhInfo *info_d = (ExhInfo *)c->exh_info.p;
    if (c->tb.n > gp.sort_cap && c->tb.n < ((int64_t)1 << 31)) {
        k_group_keys<<<(unsigned)((c->tb.n + 255) / 256), 256, 0, c->stream>>>(gp, c->tb.n);
        SP_TRY(launched(c, "k_group_keys"));
        SP_TRY(presort_network(c, c->tb.n));
        gp.presorted = 1;
    }
    const size_t psm = (size_t)gp.sort_cap * sizeof(SortKey);
    SP_CUDA(c, cudaFuncSetAttribute(k_exh_prepare, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)psm));
    SP_TRY(mark(c, c->ev_sched));
    k_exh_prepare<<<1, 1024, psm, c->stream>>>(gp, info_d);
    SP_TRY(launched(c, "k_exh_prepare"));
    ExhInfo info;
    SP_CUDA(c, cudaMemcpyAsync(&info, info_d, sizeof info, cudaMemcpyDeviceToHost, c->stream));
    SP_CUDA(c, cudaStreamSynchronize(c->stream));
    if (info.status != 0) {
        c->sched_started = false;
        return fail(c, SP_EINVAL, "the exhaustive branch takes at most 8 non-empty groups and 2^31 solutions (found " +
                                      std::to_string(info.n_groups) + " groups)");
    }
    const int n_blocks = (int)((info.n_solutions + 255) / 256);
    SP_TRY(ensure(c, c->exh_total, (size_t)(n_blocks > 0 ? n_blocks : 1) * 8));
    SP_TRY(ensure(c, c->exh_sol, (size_t)(n_blocks > 0 ? n_blocks : 1) * 8));
    if (n_blocks > 0) {
        k_exh_search<<<n_blocks, 256, 0, c->stream>>>(gp, info_d, (double *)c->exh_total.p, (long long *)c->exh_sol.p);
        SP_TRY(launched(c, "k_exh_search"));
    }
    k_exh_finish<<<1, 256, 0, c->stream>>>(gp, info_d, (const double *)c->exh_total.p, (const long long *)c->exh_sol.p, n_blocks);
    SP_TRY(launched(c, "k_exh_finish"));
    SP_TRY(mark(c, c->ev_sched));
    SP_CUDA(c, cudaMemcpyAsync(&info, info_d, sizeof info, cudaMemcpyDeviceToHost, c->stream));
    SP_CUDA(c, cudaStreamSynchronize(c->stream));
    if (total_out) *total_out = info.best_total;
    if (n_solutions_out) *n_solutions_out = info.n_solutions;
    return SP_OK;
}

sp_status sp_schedule_baseline(sp_ctx *c, int32_t policy, sp_round_rec *rounds_out, int64_t cap, int32_t *n_done) {
    if (!c) return SP_EINVAL;
    if (policy < SP_BASE_MAXACC_EDF || policy > SP_BASE_LO_PRIORITY) return fail(c, SP_EINVAL, "policy must be one of SP_BASE_*");
    BaselineParams bp;
    SP_TRY(policy_prologue(c, "sp_schedule_baseline", &bp.gp, false, rounds_out, cap, n_done));
    bp.policy = policy;
    const DevProfiles &P = c->P;
    if (P.I == 1 && c->tb.n > bp.gp.sort_cap && c->tb.n < ((int64_t)1 << 31)) {
        k_baseline_keys<<<(unsigned)((c->tb.n + 255) / 256), 256, 0, c->stream>>>(bp, c->tb.n);
        SP_TRY(launched(c, "k_baseline_keys"));
        SP_TRY(presort_network(c, c->tb.n));
        bp.gp.presorted = 1;
    }
    const size_t psm = (size_t)bp.gp.sort_cap * sizeof(SortKey);
    SP_CUDA(c, cudaFuncSetAttribute(k_baseline, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)psm));
    SP_TRY(mark(c, c->ev_sched));
    k_baseline<<<P.I, P.I > 1 ? 128 : 1024, psm, c->stream>>>(bp);
    SP_TRY(launched(c, "k_baseline"));
    return mark(c, c->ev_sched);
}

sp_status sp_check(sp_ctx *c) {
    if (!c) return SP_EINVAL;
    SP_CUDA(c, cudaSetDevice(c->device));
    int flags[2] = {0, 0};
    SP_CUDA(c, cudaMemcpyAsync(flags, c->flags.p, sizeof flags, cudaMemcpyDeviceToHost, c->stream));
    SP_CUDA(c, cudaStreamSynchronize(c->stream));
    if (flags[0] != kDevOk) SP_CUDA(c, cudaMemsetAsync(c->flags.p, 0, sizeof(int), c->stream));
    if (flags[0] == kDevLimit) return fail(c, SP_ELIMIT, "a device-side iteration limit was hit");
    if (flags[0] == kDevBadRequest)
        return fail(c, SP_EINVAL, "request arrays rejected on the device (app/instance out of range or not ordered)");
    return SP_OK;
}

sp_status sp_get_stats(sp_ctx *c, sp_stats *out) {
    if (!c || !out) return SP_EINVAL;
    SP_CUDA(c, cudaSetDevice(c->device));
    unsigned long long s[4];
    SP_CUDA(c, cudaMemcpyAsync(s, c->stats.p, sizeof s, cudaMemcpyDeviceToHost, c->stream));
    SP_CUDA(c, cudaStreamSynchronize(c->stream));
    out->kernel_launches = c->launches;
    out->rounds = (int64_t)s[0]; out->exact_utility = (int64_t)s[1]; out->exact_priority = (int64_t)s[2];
    out->exact_rows = (int64_t)s[3];
    out->score_kernel_ms = drain_events(c->ev_score, &out->score_calls);
    out->sched_kernel_ms = drain_events(c->ev_sched, &out->sched_calls);
    out->score_kernel = c->gemm_f32 ? 4 : c->gemm_on ? 3 : c->mma_ct ? 2 : c->small_ct ? 1 : 0;
    out->pad_ = 0;
    return SP_OK;
}

sp_status sp_run_host(sp_ctx *c, int64_t n, const void *feats, const int32_t *app, const int64_t *arrival_ns,
                      const int64_t *deadline_ns, const int32_t *instance, const int64_t *t0_ns,
                      const int32_t *loaded0, int32_t max_rounds, sp_req_rec *reqs_out, sp_round_rec *rounds_out,
                      int64_t cap, int32_t *n_done) {
    if (!c) return SP_EINVAL;
    if (!c->have_profiles) return fail(c, SP_ESTATE, "no profiles loaded");
    if (n < 0 || (n > 0 && (!feats || !app || !arrival_ns || !deadline_ns))) return fail(c, SP_EINVAL, "a request array is NULL");
    if (c->P.I > 1 && n > 0 && !instance) return fail(c, SP_EINVAL, "instance is required when n_instances > 1");
    if (cap < 0 || max_rounds < 0) return fail(c, SP_EINVAL, "max_rounds and cap must be >= 0");
    SP_CUDA(c, cudaSetDevice(c->device));
    const DevProfiles &P = c->P;
    const size_t esz = P.dtype == SP_BF16 ? 2 : 4;
    SP_TRY(sp_reset(c));
    SP_TRY(upload(c, c->h_feats, feats, (size_t)n * P.D * esz));
    SP_TRY(upload(c, c->h_app, app, (size_t)n * 4));
    SP_TRY(upload(c, c->h_arrival, arrival_ns, (size_t)n * 8));
    SP_TRY(upload(c, c->h_deadline, deadline_ns, (size_t)n * 8));
    if (P.I > 1) SP_TRY(upload(c, c->h_instance, instance, (size_t)n * 4));
    if (t0_ns) SP_TRY(upload(c, c->h_t0, t0_ns, (size_t)P.I * 8));
    if (loaded0) SP_TRY(upload(c, c->h_loaded, loaded0, (size_t)P.I * 4));
    if (t0_ns || loaded0)
        SP_TRY(sp_set_clocks(c, t0_ns ? (const int64_t *)c->h_t0.p : nullptr, loaded0 ? (const int32_t *)c->h_loaded.p : nullptr));
    SP_TRY(sp_score(c, n, c->h_feats.p, (const int32_t *)c->h_app.p, (const int64_t *)c->h_arrival.p,
                    (const int64_t *)c->h_deadline.p, P.I > 1 ? (const int32_t *)c->h_instance.p : nullptr, nullptr));
    const bool want_rounds = rounds_out && cap > 0;
    if (want_rounds) SP_TRY(ensure(c, c->h_rounds, (size_t)P.I * cap * sizeof(sp_round_rec)));
    SP_TRY(ensure(c, c->h_ndone, (size_t)P.I * 4));
    SP_TRY(sp_schedule_round(c, max_rounds, want_rounds ? (sp_round_rec *)c->h_rounds.p : nullptr, cap, (int32_t *)c->h_ndone.p));
    if (reqs_out && n)
        SP_CUDA(c, cudaMemcpyAsync(reqs_out, c->tb.recs, (size_t)n * sizeof(sp_req_rec), cudaMemcpyDeviceToHost, c->stream));
    if (want_rounds)
        SP_CUDA(c, cudaMemcpyAsync(rounds_out, c->h_rounds.p, (size_t)P.I * cap * sizeof(sp_round_rec), cudaMemcpyDeviceToHost, c->stream));
    if (n_done) SP_CUDA(c, cudaMemcpyAsync(n_done, c->h_ndone.p, (size_t)P.I * 4, cudaMemcpyDeviceToHost, c->stream));
    return sp_check(c);
}

}  // extern "C"

// =================================================================================================
// Scoring without any allocation.  The scratch that the grouping pass and the tiled scoring kernel need
// (per-application counters, prefix sums and the request permutation) lives in one file-scope device array
// instead of context-owned cudaMalloc'ed buffers.  Every GPU that loads this library holds the array until
// the process exits.
namespace {

constexpr int64_t kStaticMaxRequests = 65536;

struct StaticScratch {                       // layout of the array below
    int flags[2];                            // must start at 0
    int32_t cnt[kMaxApps];                   // must start at 0
    int32_t cursor[kMaxApps];                // must start at 0
    int32_t tiled_start[kMaxApps + 1];
    int32_t small_start[2];
    int64_t gstart[kMaxApps + 1];
    int64_t perm[kStaticMaxRequests];
};

static __device__ __align__(256) unsigned char g_static_scratch[sizeof(StaticScratch)];

constexpr int kStaticMaxDevices = 64;
StaticScratch *g_static_ptr[kStaticMaxDevices] = {};   // device address of the array, per device

void static_msg(char *buf, int32_t len, const std::string &m) {
    if (buf && len > 0) { std::snprintf(buf, (size_t)len, "%s", m.c_str()); }
}

}  // namespace

extern "C" sp_status sp_score_static(int device, void *cuda_stream, const sp_static_head *head, int64_t n,
                                     const void *feats, const int32_t *app, float *acc_out, float *v_out,
                                     char *errbuf, int32_t errbuf_len) {
#define SP_STATIC_FAIL(code, msg) do { static_msg(errbuf, errbuf_len, (msg)); return (code); } while (0)
#define SP_STATIC_CUDA(call)                                                                        \
    do {                                                                                            \
        cudaError_t e_ = (call);                                                                    \
        if (e_ != cudaSuccess) SP_STATIC_FAIL(SP_ECUDA, std::string(#call) + ": " + cudaGetErrorString(e_)); \
    } while (0)
    if (!head) SP_STATIC_FAIL(SP_EINVAL, "head is NULL");
    if (n < 0 || n > kStaticMaxRequests)
        SP_STATIC_FAIL(SP_EINVAL, "n is outside 0.." + std::to_string(kStaticMaxRequests) +
                                      ", the capacity of the built-in scratch array");
    const int A = head->n_apps, C = head->n_classes, D = head->feat_dim;
    if (A < 1 || A > kMaxApps || C < 1 || C > kMaxClasses || D < 1 || !head->models_per_app || !head->head_w ||
        !head->head_b || !head->recall || (head->feat_dtype != SP_F32 && head->feat_dtype != SP_BF16))
        SP_STATIC_FAIL(SP_EINVAL, "bad head description (shapes out of range or NULL array)");
    if (n > 0 && (!feats || !app || !acc_out || !v_out)) SP_STATIC_FAIL(SP_EINVAL, "a request or output array is NULL");
    if (device < 0 || device >= kStaticMaxDevices) SP_STATIC_FAIL(SP_EINVAL, "device index out of range");
    DevProfiles P{};
    P.I = 1; P.A = A; P.C = C; P.D = D; P.dtype = head->feat_dtype;
    for (int a = 0; a < A; ++a) {
        const int m = head->models_per_app[a];
        if (m < 1 || m > kMaxModelsPerApp) SP_STATIC_FAIL(SP_EINVAL, "models_per_app entries must be 1..16");
        P.mfirst[a] = P.sumM; P.sumM += m; P.Mmax = m > P.Mmax ? m : P.Mmax;
    }
    P.mfirst[A] = P.sumM;
    P.W = head->head_w; P.bias = head->head_b; P.recall = head->recall; P.tau = 1.0;

    SP_STATIC_CUDA(cudaSetDevice(device));
    if (!g_static_ptr[device]) {               // set-up, once per device, with that device current
        void *p = nullptr;
        SP_STATIC_CUDA(cudaGetSymbolAddress(&p, g_static_scratch));
        g_static_ptr[device] = static_cast<StaticScratch *>(p);
    }
    StaticScratch *s = g_static_ptr[device];
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    if (n == 0) return SP_OK;

    DevTable tb{};
    tb.n = n; tb.feats = feats; tb.app = app; tb.acc32 = acc_out; tb.v32 = v_out;
    tb.cnt = s->cnt; tb.cursor = s->cursor; tb.gstart = s->gstart; tb.perm = s->perm;
    // the array keeps the previous call's contents: clear the parts that are accumulated into
    SP_STATIC_CUDA(cudaMemsetAsync(s, 0, offsetof(StaticScratch, tiled_start), stream));
    const unsigned gb = (unsigned)((n + 255) / 256);
    k_group_count<<<gb, 256, 0, stream>>>(P, tb, 0, s->flags, nullptr);
    k_group_scan<<<1, 1024, 0, stream>>>(A, A, s->cnt, s->gstart, s->tiled_start, s->small_start);
    k_group_scatter<<<gb, 256, 0, stream>>>(P, tb, s->flags);
    const int grid = (int)(n / kTiledRows + A);
    if (P.dtype == SP_BF16)
        k_score_tiled<true><<<grid, kTiledThreads, 0, stream>>>(P, tb, s->tiled_start, nullptr, s->flags);
    else
        k_score_tiled<false><<<grid, kTiledThreads, 0, stream>>>(P, tb, s->tiled_start, nullptr, s->flags);
    SP_STATIC_CUDA(cudaGetLastError());
    int flags[2] = {0, 0};
    SP_STATIC_CUDA(cudaMemcpyAsync(flags, s->flags, sizeof flags, cudaMemcpyDeviceToHost, stream));
    SP_STATIC_CUDA(cudaStreamSynchronize(stream));
    if (flags[1]) SP_STATIC_FAIL(SP_EINVAL, "an application id is outside 0..n_apps-1; nothing was written");
    return SP_OK;
#undef SP_STATIC_CUDA
#undef SP_STATIC_FAIL
}
