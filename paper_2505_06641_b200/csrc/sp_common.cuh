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

// The request table: caller-owned inputs (borrowed) + context-owned results.
struct DevTable {
    int64_t n;
    const void *feats;
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
    int64_t *gstart;             // [I*A+1] exclusive prefix of cnt == start of each queue region
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

__device__ __forceinline__ void dev_error(int *status, int code) { atomicMax(status, code); }

}  // namespace sp
