// Multi-block sort of a large snapshot queue.
//
// k_sched sorts the requests that join an instance's queues with one thread block.  That is right for the few
// arrivals of a round, but a single-instance snapshot of tens of thousands of requests (all pending at once) would
// spend milliseconds in that one block.  These kernels sort the keys (application, deadline, index) of such an
// instance with the whole GPU before k_sched starts, into the scratch array k_sched would have sorted itself:
// the same bitonic network with ascending comparators only (a partner index >= n stands for +infinity, so n needs
// no padding), steps whose partners lie inside a 4,096-key chunk run in shared memory, the others one launch each.
#pragma once

#include "sp_common.cuh"
#include "sp_sched.cuh"

namespace sp {

constexpr int kPresortChunk = 4096;       // keys per block in shared memory (64 KB)
constexpr int kPresortThreads = 1024;

__global__ void k_presort_keys(DevTable tb, SortKey *keys, int64_t n) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    SortKey k; k.dl = tb.deadline[i]; k.id_rel = (int32_t)i; k.app = tb.app[i];
    keys[i] = k;
}

// One compare-exchange of the network for the pair with low index i (bit j clear) at merge size k.
__device__ __forceinline__ void presort_pair(SortKey *keys, int64_t base, int64_t n, int64_t i, int64_t j, int64_t k) {
    const int64_t partner = (j == (k >> 1)) ? (i ^ (k - 1)) : (i ^ j);
    if (partner < n && i < n) {
        const SortKey a = keys[i - base], b = keys[partner - base];
        if (key_less(b, a)) { keys[i - base] = b; keys[partner - base] = a; }
    }
}

// All steps with partners inside the block's chunk: for merge sizes k_from .. k_to (each from j = min(k / 2, chunk / 2)
// down to 1).  k_from = 2 sorts the chunk; k_from = k_to > chunk finishes a merge whose wide steps ran globally.
__global__ void __launch_bounds__(kPresortThreads) k_presort_local(SortKey *keys, int64_t n, int64_t k_from, int64_t k_to) {
    extern __shared__ __align__(16) unsigned char dyn[];
    SortKey *s = reinterpret_cast<SortKey *>(dyn);
    const int64_t base = (int64_t)blockIdx.x * kPresortChunk;
    for (int t = threadIdx.x; t < kPresortChunk; t += kPresortThreads)
        if (base + t < n) s[t] = keys[base + t];
    __syncthreads();
    for (int64_t k = k_from; k <= k_to; k <<= 1) {
        for (int64_t j = (k >> 1) < kPresortChunk ? (k >> 1) : (kPresortChunk >> 1); j > 0; j >>= 1) {
            if (j == (k >> 1) && k > kPresortChunk) continue;      // the mirrored first step of a wide merge ran globally
            for (int t = threadIdx.x; t < (kPresortChunk >> 1); t += kPresortThreads) {
                const int64_t tt = (base >> 1) + t;                // global pair number
                const int64_t i = ((tt & ~(j - 1)) << 1) | (tt & (j - 1));
                presort_pair(s, base, n, i, j, k);
            }
            __syncthreads();
        }
    }
    for (int t = threadIdx.x; t < kPresortChunk; t += kPresortThreads)
        if (base + t < n) keys[base + t] = s[t];
}

// One step (k, j) whose partners are further apart than a chunk.
__global__ void k_presort_global(SortKey *keys, int64_t n, int64_t k, int64_t j, int64_t n_pairs) {
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= n_pairs) return;
    const int64_t i = ((t & ~(j - 1)) << 1) | (t & (j - 1));
    presort_pair(keys, 0, n, i, j, k);
}

}  // namespace sp
