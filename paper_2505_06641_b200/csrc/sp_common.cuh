// Shared device-side definitions of the scoring-and-selection library (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "../../include/sneakpeek.h"

namespace sp {

constexpr int kMaxApps = 16;          // applications per instance
constexpr int kMaxModelsPerApp = 16;  // model variants per application
constexpr int kMaxBatchSizes = 16;
constexpr int kMaxBatch = 1024;       // largest allowed batch size
constexpr int kMaxClasses = 4096;

// Errors recorded on the device (combined with atomicMax; larger = reported first).
enum DevErr : int { kDevOk = 0, kDevBadRequest = 1, kDevLimit = 2 };

// Profiles as the kernels see them (passed by value).
struct DevProfiles {
    int I, A, C, D, dtype, sumM, Mmax, nB;
    const void *W;            // [I][A][D][C]
    const float *bias;        // [I][A][C]
    const float *recall;      // [I][sumM][C]
    const float *prior;       // [I][A][C] or nullptr
    const float *prior_dot;   // [I][sumM]  sum_c alpha_c * recall[m][c]   (nullptr without prior)
    const float *prior_sum;   // [I][A]     sum_c alpha_c
    float kappa;
    const int64_t *lat_alpha, *lat_beta, *swap;   // [I][sumM]
    double tau;
    int mfirst[kMaxApps + 1];  // first global model id of each application
    int batch[kMaxBatchSizes];
    int pen[kMaxApps];         // penalty of Eq. 2 per application (SP_PEN_*)
    int any_soft;              // some application has a penalty other than the step
};

// One sp_score() call's feature matrix: rows [first, next segment's first) of the request table live in `feats`.
struct FeatSeg { int64_t first; const void *feats; };

// The request table: caller-owned inputs (borrowed) + context-owned results.
struct DevTable {
    int64_t n;
    const void *feats;           // feature matrix of the table; nullptr once requests were appended (see segs)
    const FeatSeg *segs;         // after an append: the feature matrices of the calls, ascending by first row
    int n_segs;
    const int32_t *app;
    const int64_t *arrival, *deadline;
    const int32_t *instance;     // nullptr when I == 1
    float *acc32;                // [n][Mmax]
    float *v32;                  // [n]
    double *acc64;               // [n][Mmax]  filled on demand by the fp64 re-evaluation
    double *v64;                 // [n]
    unsigned char *exact;        // [n] 1 when acc64/v64 hold this row
    sp_req_rec *recs;            // [n]
    int32_t *cnt;                // [I*A]   requests per (instance, application)
    int64_t *gstart;             // [I*A+1] exclusive prefix of cnt (grouping of the rows scored by one call)
    const int64_t *qstart;       // [I*A+1] start of each (instance, application) queue region; equals gstart until requests are appended
    int64_t *perm;               // [n] request ids grouped by (instance, application)
    int32_t *cursor;             // [I*A] scratch of the grouping pass
};

__device__ __forceinline__ float bf16_bits_to_float(unsigned short b) {
    return __uint_as_float(((unsigned int)b) << 16);
}

__device__ __forceinline__ float load_feat(const void *base, int dtype, int64_t idx) {
    return dtype == SP_BF16 ? bf16_bits_to_float(((const unsigned short *)base)[idx])
                            : ((const float *)base)[idx];
}

// Feature row of request `id`: base pointer of its matrix and the row index inside it.
__device__ __forceinline__ const void *feat_matrix(const DevTable &tb, int64_t id, int64_t &row) {
    if (tb.feats) { row = id; return tb.feats; }
    int lo = 0, hi = tb.n_segs - 1;                      // last segment whose first row is <= id
    while (lo < hi) { const int mid = (lo + hi + 1) >> 1; if (tb.segs[mid].first <= id) lo = mid; else hi = mid - 1; }
    row = id - tb.segs[lo].first;
    return tb.segs[lo].feats;
}

__device__ __forceinline__ void dev_error(int *status, int code) { atomicMax(status, code); }

}  // namespace sp
