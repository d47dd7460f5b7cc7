// Grouping pass of sp_score(): validates the request arrays and counts / orders requests by
// (instance, application).  The counts size every application's queue region; the permutation
// feeds the tiled scoring kernel, which needs tiles of requests that share one head.
#pragma once

#include "sp_common.cuh"

namespace sp {

constexpr int kTiledRows = 64;    // requests per tile of the tiled scoring kernel
constexpr int kSmallRows = 128;   // requests per tile of the small-head scoring kernel

// Validation of the request table, initial request records, requests per (instance, application).
// flags[0]: device status (DevErr), flags[1]: 1 when the request table failed validation.
// prev_arrival: arrival time of the last request already in the table when these rows are appended to it (nullptr
// for the first rows of a table); in trace mode the appended rows must not arrive before it.
__global__ void k_group_count(DevProfiles P, DevTable tb, int trace_mode, int *flags, const int64_t *prev_arrival) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= tb.n) return;
    if (tb.recs) {                           // the request starts pending, without an fp64 re-scoring (a table
        sp_req_rec r; r.status = SP_PENDING; r.round = -1; r.model = -1; r.worker = 0; r.order = 0;   // that is only scored has no records)
        tb.recs[i] = r;
        tb.exact[i] = 0;
    }
    const int a = tb.app[i];
    const int inst = tb.instance ? tb.instance[i] : 0;
    bool bad = a < 0 || a >= P.A || inst < 0 || inst >= P.I;
    if (!bad && i == 0 && trace_mode && prev_arrival && *prev_arrival > tb.arrival[0]) bad = true;
    if (!bad && i > 0) {
        const int prev = tb.instance ? tb.instance[i - 1] : 0;
        if (prev > inst) bad = true;
        if (trace_mode && prev == inst && tb.arrival[i - 1] > tb.arrival[i]) bad = true;
    }
    if (bad) {
        dev_error(&flags[0], kDevBadRequest);
        flags[1] = 1;
        return;
    }
    const int key = inst * P.A + a;
    // one atomic per distinct key in the warp
    const unsigned peers = __match_any_sync(__activemask(), key);
    if ((int)(__ffs(peers) - 1) == (int)(threadIdx.x & 31)) atomicAdd(&tb.cnt[key], __popc(peers));
}

// Single block.  gstart = exclusive prefix of cnt (int64); tiled_start = exclusive prefix of
// ceil(cnt / kTiledRows) per (instance, app); small_start = exclusive prefix over instances of
// ceil(requests of the instance / kSmallRows).
__global__ void __launch_bounds__(1024) k_group_scan(int n_keys, int A, const int32_t *cnt, int64_t *gstart,
                                                     int32_t *tiled_start, int32_t *small_start) {
    __shared__ long long warp_sum[32];
    __shared__ long long carry[3];
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    if (tid < 3) carry[tid] = 0;
    __syncthreads();
    // pass 0: gstart, pass 1: tiled tiles, pass 2: small tiles (over instances)
    for (int pass = 0; pass < 3; ++pass) {
        const int len = pass == 2 ? n_keys / A : n_keys;
        for (int base = 0; base < len; base += 1024) {
            const int k = base + tid;
            long long val = 0;
            if (k < len) {
                if (pass == 0) val = cnt[k];
                else if (pass == 1) val = (cnt[k] + kTiledRows - 1) / kTiledRows;
                else {
                    long long s = 0;
                    for (int a = 0; a < A; ++a) s += cnt[k * A + a];
                    val = (s + kSmallRows - 1) / kSmallRows;
                }
            }
            long long incl = val;
            for (int o = 1; o < 32; o <<= 1) {
                const long long t = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += t;
            }
            if (lane == 31) warp_sum[wid] = incl;
            __syncthreads();
            if (wid == 0) {
                long long w = warp_sum[lane];
                for (int o = 1; o < 32; o <<= 1) {
                    const long long t = __shfl_up_sync(0xffffffffu, w, o);
                    if (lane >= o) w += t;
                }
                warp_sum[lane] = w;
            }
            __syncthreads();
            const long long excl = carry[pass] + (wid ? warp_sum[wid - 1] : 0) + incl - val;
            if (k < len) {
                if (pass == 0) gstart[k] = excl;
                else if (pass == 1) tiled_start[k] = (int32_t)excl;
                else small_start[k] = (int32_t)excl;
            }
            __syncthreads();
            if (tid == 0) carry[pass] += warp_sum[31];
            __syncthreads();
        }
        if (tid == 0) {
            if (pass == 0) gstart[len] = carry[0];
            else if (pass == 1) tiled_start[len] = (int32_t)carry[1];
            else small_start[len] = (int32_t)carry[2];
        }
        __syncthreads();
    }
}

// Multi-block version of k_group_scan for many (instance, application) keys: block b owns keys (and instances)
// [1024 b, 1024 b + 1024).  First kernel: per-block totals of the three scanned quantities; second kernel: every
// block adds up the totals of the blocks before it and scans its own chunk.
constexpr int kScanChunk = 1024;

__device__ __forceinline__ long long scan_value(int pass, int k, int len, int A, const int32_t *cnt) {
    if (k >= len) return 0;
    if (pass == 0) return cnt[k];
    if (pass == 1) return (cnt[k] + kTiledRows - 1) / kTiledRows;
    long long s = 0;
    for (int a = 0; a < A; ++a) s += cnt[(int64_t)k * A + a];
    return (s + kSmallRows - 1) / kSmallRows;
}

__device__ __forceinline__ long long block_reduce_ll(long long v, long long *warp_sum) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();
    if (lane == 0) warp_sum[wid] = v;
    __syncthreads();
    long long w = lane < (int)(blockDim.x >> 5) ? warp_sum[lane] : 0;
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) w += __shfl_xor_sync(0xffffffffu, w, o);
    return w;                                           // valid in every thread
}

__global__ void __launch_bounds__(kScanChunk) k_group_partials(int n_keys, int A, const int32_t *cnt, long long *partial) {
    __shared__ long long warp_sum[32];
    const int k = blockIdx.x * kScanChunk + threadIdx.x, nblk = gridDim.x;
    for (int pass = 0; pass < 3; ++pass) {
        const long long t = block_reduce_ll(scan_value(pass, k, pass == 2 ? n_keys / A : n_keys, A, cnt), warp_sum);
        if (threadIdx.x == 0) partial[pass * nblk + blockIdx.x] = t;
    }
}

__global__ void __launch_bounds__(kScanChunk)
k_group_scan_blocks(int n_keys, int A, const int32_t *cnt, const long long *partial, int64_t *gstart,
                    int32_t *tiled_start, int32_t *small_start) {
    __shared__ long long warp_sum[32];
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5, nblk = gridDim.x;
    const int k = blockIdx.x * kScanChunk + tid;
    for (int pass = 0; pass < 3; ++pass) {
        const int len = pass == 2 ? n_keys / A : n_keys;
        long long before = 0;
        for (int b = tid; b < (int)blockIdx.x; b += kScanChunk) before += partial[pass * nblk + b];
        before = block_reduce_ll(before, warp_sum);
        const long long val = scan_value(pass, k, len, A, cnt);
        long long incl = val;
        for (int o = 1; o < 32; o <<= 1) {
            const long long t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        __syncthreads();
        if (lane == 31) warp_sum[wid] = incl;
        __syncthreads();
        if (wid == 0) {
            long long w = warp_sum[lane];
            for (int o = 1; o < 32; o <<= 1) {
                const long long t = __shfl_up_sync(0xffffffffu, w, o);
                if (lane >= o) w += t;
            }
            warp_sum[lane] = w;
        }
        __syncthreads();
        const long long excl = before + (wid ? warp_sum[wid - 1] : 0) + incl - val;
        if (k <= len) {                                 // k == len: the grand total (the element past the end)
            if (pass == 0) gstart[k] = excl;
            else if (pass == 1) tiled_start[k] = (int32_t)excl;
            else small_start[k] = (int32_t)excl;
        }
        __syncthreads();
    }
}

__global__ void k_group_scatter(DevProfiles P, DevTable tb, const int *flags) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= tb.n || flags[1]) return;
    const int key = (tb.instance ? tb.instance[i] : 0) * P.A + tb.app[i];
    const int pos = atomicAdd(&tb.cursor[key], 1);
    tb.perm[tb.gstart[key] + pos] = i;
}

}  // namespace sp
