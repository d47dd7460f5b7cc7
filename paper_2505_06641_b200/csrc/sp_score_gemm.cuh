// Tensor-core scoring kernel for large heads (the head is a real GEMM: thousands of requests x hundreds of
// labels x D up to thousands), in two flavours: bf16 features and weights, and fp32 features and weights.
//
// Per request (Section 4.1 + Eq. 9 + Eq. 12 of the paper):
//   z = x W_a + b_a;  p = softmax(z);  theta = Dirichlet posterior mean;  acc_j = sum_c theta_c recall_j(c);
//   v = 1 + population variance_j(acc_j).
// Shape of the computation: a tile is 128 requests of one (instance, application) group (gathered through the
// grouping permutation), the labels are swept in chunks of NC logit columns, and for every chunk the logits
// Z[128 x NC] = X[128 x D] W^T[NC x D]^T accumulate over 128-byte feature slabs in tensor memory (tcgen05 MMAs,
// operands K-major with 128-byte swizzle).  Neither logits nor posterior leave the SM: epilogue warps read each
// finished chunk from tensor memory and fold it into an online softmax (running max, running sum) with the recall
// contraction fused (running sum of 2^z * recall_j), flash-attention style; the two accumulators alternate so the
// epilogue of a chunk overlaps the MMAs of the next one.
//   * A operand: requests of a group are not contiguous, so 4 producer warps gather their rows with 16-byte
//     cp.async copies into the swizzled slab.  Eight consecutive lanes copy the eight 16-byte pieces of one row's
//     128 bytes, so every warp instruction asks for four whole 128-byte lines (one lane per row, eight instructions
//     each touching 32 different lines, measured 1.8 x slower on the 2 GB trace workload and 1.3 x on C3).
//   * B operand: the head is transposed once, when the profiles are loaded, into a K-major image
//     Wt[(instance, application, label)][feature]; TMA tiles of NC labels x one slab of features stream from it
//     (L2 resident).  The chunk's recall rows and bias arrive by TMA as well.
//   * bf16: NC = 256, 64 features per slab, one MMA pass (bf16 products are exact in the fp32 accumulator).
//   * fp32: NC = 208, 32 features per slab, tf32 MMAs with the split x = x_hi + x_lo, W = W_hi + W_lo (hi = value
//     truncated to tf32, lo = exact remainder): x_hi W_hi + x_hi W_lo + x_lo W_hi, the dropped term is below 2^-20
//     relative.  The image holds W_hi and W_lo (log2(e) folded in); x_hi is the gathered slab as it is (the unit
//     reads the truncated value), x_lo is computed by the producer threads from their own row and stored into a
//     32-column slot of tensor memory, from where the third MMA takes its A operand.
//   * Epilogue: 2 groups of 4 warps split the columns of a chunk; each keeps its own running state for the row and
//     the two are merged at the end of the tile.
// Every wait on an mbarrier is bounded; when one runs out the block raises kDevLimit and leaves.
#pragma once

#include <cuda.h>

#include "sp_common.cuh"
#include "sp_score_mma.cuh"   // mbarrier / TMA / tcgen05 helpers

namespace sp {
namespace gemm {

using namespace sp::mma;

constexpr int kGRows = 128;                 // requests per tile = MMA M
constexpr int kASlabBytes = kGRows * 128;   // 16 KB: 128 rows x 128 bytes
constexpr int kGBProducerWarp = 0, kGMmaWarp = 1, kGAWarp0 = 2, kGEpiWarp0 = 6;
constexpr int kGAThreads = 128;
constexpr int kGMaxEpiGroups = 4;
constexpr int kMergeFloats = 2 + kMaxModelsPerApp;    // running max, running sum, running sums per model
constexpr int kGMaxA = 5, kGMaxB = 3;      // largest A / B ring of the two flavours

// Two fp32 values in one 64-bit register for the two-wide FP32 instructions.
__device__ __forceinline__ unsigned long long pack_f32x2(float lo, float hi) {
    unsigned long long v;
    asm("mov.b64 %0, {%1, %2};" : "=l"(v) : "f"(lo), "f"(hi));
    return v;
}
// acc = a * b + acc on both halves (round to nearest, one instruction).
__device__ __forceinline__ void fma_f32x2(unsigned long long &acc, unsigned long long a, unsigned long long b) {
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(acc) : "l"(a), "l"(b));
}
__device__ __forceinline__ float sum_f32x2(unsigned long long v) {
    float lo, hi;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
    return lo + hi;
}

template <bool F32>
struct GCfg {
    // Epilogue warpgroups (each takes an equal share of the columns of every chunk) and the logit columns a thread
    // holds in registers at a time.  Measured: the fp32 flavour is 14 % faster with four groups (its chunk has to be
    // finished while only three operand slabs are in flight), the bf16 flavour 2 % slower than with two.
    static constexpr int EpiGroups = F32 ? 4 : 2;
    static constexpr int EpiBlk = F32 ? 16 : 32;
    static constexpr int EpiThreads = 128 * EpiGroups;
    static constexpr int Threads = 32 * 6 + EpiThreads;
    static constexpr int NC = F32 ? 208 : 256;                 // logit columns per chunk = MMA N (2 accumulators <= 512 columns)
    static constexpr int KSlab = F32 ? 32 : 64;                // features per slab row (128 bytes)
    static constexpr int KStep = F32 ? 8 : 16;                 // features per MMA
    static constexpr int BSlabBytes = NC * 128 * (F32 ? 2 : 1);   // fp32: W_hi rows, then W_lo rows
    static constexpr int BSlot = (BSlabBytes + 1023) & ~1023;
    // The A slabs are gathered by threads (cp.async) and need several slabs in flight to cover the L2 latency; the B
    // slabs come by TMA.  Separate rings let the small A slabs (16 KB) run deeper than the large B slabs.
    static constexpr int AStages = F32 ? 3 : 5;                // fp32: one x_lo slot of tensor memory per A stage (3 x 32 columns)
    static constexpr int BStages = F32 ? 2 : 3;
    // A slab is reported complete when ADepth newer slabs have been issued (cp.async completion is observed relative
    // to newer groups); issuing needs free slots, so the ring is deeper than ADepth by the slabs the MMAs work on.
    static constexpr int ADepth = F32 ? 1 : 2;
    static constexpr int RBytes = kMaxModelsPerApp * NC * 4;   // recall rows of a chunk
    static constexpr int BiasBytes = NC * 4;
    static constexpr int BiasSlot = (BiasBytes + 127) & ~127;     // TMA destinations are 128-byte aligned
    static_assert(RBytes % 128 == 0, "recall buffers must keep the 128-byte alignment of TMA destinations");
    static_assert(AStages <= kGMaxA && BStages <= kGMaxB, "the barrier table holds kGMaxA / kGMaxB stages");
    static constexpr int TmemLo = 2 * NC;                      // fp32: x_lo slots (32 columns per stage) after the accumulators
    // byte offsets from the 1024-byte aligned base
    static constexpr int a_ring = 0;                                          // [AStages] slabs of 128 rows
    static constexpr int b_ring = a_ring + AStages * kASlabBytes;             // [BStages] slabs of NC (x 2) rows
    static constexpr int rtab = b_ring + BStages * BSlot;                     // [2][16][NC] floats
    static constexpr int bias = rtab + 2 * RBytes;                            // [2][NC] floats
    static constexpr int merge = bias + 2 * BiasSlot;                        // [EpiGroups - 1][128][kMergeFloats]
    static constexpr int bars = (merge + (EpiGroups - 1) * kGRows * kMergeFloats * 4 + 15) & ~15;
    static constexpr int n_bars = 3 * kGMaxA + 2 * kGMaxB + 8 + 3;
    static constexpr int misc = bars + n_bars * 8;
    static constexpr int end = misc + 16;
    static constexpr int bytes = end + 1024;
};
__device__ __forceinline__ constexpr int gbar_full_a(int s) { return s; }
__device__ __forceinline__ constexpr int gbar_free_a(int s) { return kGMaxA + s; }
__device__ __forceinline__ constexpr int gbar_full_b(int s) { return 2 * kGMaxA + s; }
__device__ __forceinline__ constexpr int gbar_free_b(int s) { return 2 * kGMaxA + kGMaxB + s; }
constexpr int kGBar2 = 2 * kGMaxA + 2 * kGMaxB;
__device__ __forceinline__ constexpr int gbar_acc_full(int b) { return kGBar2 + b; }
__device__ __forceinline__ constexpr int gbar_acc_empty(int b) { return kGBar2 + 2 + b; }
__device__ __forceinline__ constexpr int gbar_r_full(int b) { return kGBar2 + 4 + b; }
__device__ __forceinline__ constexpr int gbar_r_free(int b) { return kGBar2 + 6 + b; }
constexpr int kGBarMergeReady = kGBar2 + 8;
constexpr int kGBarMergeDone = kGBar2 + 9;
constexpr int kGBarDrain = kGBar2 + 10;
// fp32: every producer thread's copies of A stage s have landed (the threads then read rows other threads copied)
__device__ __forceinline__ constexpr int gbar_landed(int s) { return kGBar2 + 11 + s; }

struct GParams {
    DevProfiles P;
    DevTable tb;
    const int4 *tiles;       // (key = instance * A + application, first position in perm, rows, -); key -1 = unused entry
    int n_tiles;
    int Cp;                  // labels per application in the transposed head image (C rounded up to 16)
    int lo_row0;             // fp32: first row of the W_lo half of the image (= number of W_hi rows)
    float *acc_out;
    int *flags;
    // Work items.  split = 1: an item is a tile.  split = 2: an item is half of a tile's label chunks, so that a launch
    // of few tiles per block still spreads evenly (512 tiles on 148 blocks: 4 tiles on the busiest block, but 7 of 1,024
    // halves); the two halves of a row meet in global memory: each writes its running (maximum, sum, sums per model) to
    // `partial`, and the one that comes second (per-row counter `part_count`, zeroed before the launch) merges and stores.
    int split;
    float *partial;          // [n_tiles][2][kMergeFloats][128]
    int *part_count;         // [n_tiles][128]
};

// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = n.
__host__ __device__ constexpr uint32_t instr_desc_bf16(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kGRows >> 4) << 24);
}
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n.reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc)
        : "memory");
}
// 16-byte async copy that reads only src_bytes (0..16) from global memory and fills the rest with zeros.
__device__ __forceinline__ void cp_async16_zfill(uint32_t dst, const void *src, uint32_t src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Transposes the heads into the K-major image Wt[(i * A + a) * Cp + c][d] (bf16 bit patterns), labels c >= C zero.
__global__ void k_transpose_head_bf16(const unsigned short *__restrict__ W, unsigned short *__restrict__ Wt, int64_t n_heads,
                                      int D, int C, int Cp) {
    __shared__ unsigned short tile[32][33];
    const int64_t head = blockIdx.z;
    const int d0 = blockIdx.y * 32, c0 = blockIdx.x * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;          // 32 x 8 threads
    for (int r = ty; r < 32; r += 8) {
        const int d = d0 + r, c = c0 + tx;
        tile[r][tx] = (d < D && c < C) ? W[(head * D + d) * C + c] : (unsigned short)0;
    }
    __syncthreads();
    for (int r = ty; r < 32; r += 8) {
        const int c = c0 + r, d = d0 + tx;
        if (c < Cp && d < D) Wt[(head * Cp + c) * D + d] = tile[tx][r];
    }
}

// fp32 heads: K-major images of W * log2(e) split for the tf32 unit: rows [0, n_heads * Cp) hold the value truncated to
// tf32, rows [n_heads * Cp, 2 n_heads * Cp) the exact remainder; labels c >= C zero.
__global__ void k_transpose_head_f32(const float *__restrict__ W, float *__restrict__ Wt, int64_t n_heads, int D, int C, int Cp) {
    __shared__ float tile[32][33];
    const int64_t head = blockIdx.z;
    const int d0 = blockIdx.y * 32, c0 = blockIdx.x * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;          // 32 x 8 threads
    for (int r = ty; r < 32; r += 8) {
        const int d = d0 + r, c = c0 + tx;
        tile[r][tx] = (d < D && c < C) ? W[(head * D + d) * C + c] : 0.f;
    }
    __syncthreads();
    for (int r = ty; r < 32; r += 8) {
        const int c = c0 + r, d = d0 + tx;
        if (c < Cp && d < D) {
            const float w = tile[tx][r] * kLog2e, hi = tf32_part(w);
            Wt[(head * Cp + c) * D + d] = hi;
            Wt[((n_heads + head) * Cp + c) * D + d] = w - hi;
        }
    }
}

// Tile table: every (instance, application) group is cut into tiles of 128 requests; the order of the entries is
// arbitrary (slots are handed out by an atomic counter), unused entries keep key -1.
__global__ void k_gemm_tiles(int n_keys, const int32_t *__restrict__ cnt, const int64_t *__restrict__ gstart,
                             int4 *__restrict__ tiles, int *__restrict__ counter, const int *__restrict__ flags) {
    const int key = blockIdx.x * blockDim.x + threadIdx.x;
    if (key >= n_keys || flags[1]) return;
    const int n = cnt[key];
    if (n <= 0) return;
    const int nt = (n + kGRows - 1) / kGRows;
    const int base = atomicAdd(counter, nt);
    for (int i = 0; i < nt; ++i) {
        const int rows = n - i * kGRows < kGRows ? n - i * kGRows : kGRows;
        tiles[base + i] = make_int4(key, (int)(gstart[key] + (int64_t)i * kGRows), rows, 0);
    }
}

template <bool F32>
__global__ void __launch_bounds__(GCfg<F32>::Threads, 1)
k_score_gemm(const __grid_constant__ CUtensorMap wt_map, const __grid_constant__ CUtensorMap r_map,
             const __grid_constant__ CUtensorMap b_map, const GParams prm) {
    using G = GCfg<F32>;
    constexpr int kNC = G::NC, kKSlab = G::KSlab, kAStages = G::AStages, kBStages = G::BStages;
    constexpr int kBSlabBytes = G::BSlabBytes, kRBytes = G::RBytes, kBiasBytes = G::BiasBytes;
    constexpr int kGEpiGroups = G::EpiGroups, kGEpiBlk = G::EpiBlk, kGEpiThreads = G::EpiThreads;
    using GSmem = G;
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw_u32 = smem_u32(smem_raw);
    const uint32_t base = (raw_u32 + 1023u) & ~1023u;
    unsigned char *sm = smem_raw + (base - raw_u32);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(sm + GSmem::misc);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(sm + GSmem::misc + 4);
    auto bar = [&](int i) -> uint32_t { return base + GSmem::bars + 8u * (uint32_t)i; };

    const DevProfiles &P = prm.P;
    const DevTable &tb = prm.tb;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int A = P.A, C = P.C, D = P.D, Cp = prm.Cp;
    const int n_ks = (D + kKSlab - 1) / kKSlab;            // feature slabs
    const int n_ch = (C + kNC - 1) / kNC;                  // label chunks
    const int S = prm.split, n_items = prm.n_tiles * S;    // work items: tiles, or halves of a tile's label chunks

    if (tid == 0) {
        for (int s = 0; s < kAStages; ++s) {
            mbar_init(bar(gbar_full_a(s)), kGAThreads); mbar_init(bar(gbar_free_a(s)), 1); mbar_init(bar(gbar_landed(s)), kGAThreads);
        }
        for (int s = 0; s < kBStages; ++s) { mbar_init(bar(gbar_full_b(s)), 1); mbar_init(bar(gbar_free_b(s)), 1); }
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar(gbar_acc_full(b)), 1); mbar_init(bar(gbar_acc_empty(b)), kGEpiThreads);
            mbar_init(bar(gbar_r_full(b)), 1); mbar_init(bar(gbar_r_free(b)), kGEpiThreads);
        }
        mbar_init(bar(kGBarMergeReady), kGEpiThreads - 128);
        mbar_init(bar(kGBarMergeDone), 128);
        mbar_init(bar(kGBarDrain), 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kGMmaWarp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    if (tmem != 0 && tid == 0) *abort_flag = 1;                // cannot happen for a whole-memory allocation
    __syncthreads();
    const bool tmem_ok = *abort_flag == 0;

    if (!tmem_ok) {
        // unexpected tensor-memory base: nothing runs, the block reports the error below
    } else if (warp == kGBProducerWarp) {
        // ================================================================ TMA producer of W^T slabs, recall rows, bias
        if (lane == 0) {
            uint32_t slab_seq = 0, chunk_seq = 0;
            bool ok = true;
            for (int it = blockIdx.x; it < n_items && ok; it += gridDim.x) {
                const int t = it / S, hf = it - t * S;
                const int4 d = prm.tiles[t];
                if (d.x < 0) continue;
                const int inst = d.x / A, a = d.x - inst * A;
                const int wrow0 = d.x * Cp;                              // first row of this head in the image
                for (int ch = hf * n_ch / S; ch < (hf + 1) * n_ch / S && ok; ++ch, ++chunk_seq) {
                    const int rb = chunk_seq & 1;
                    const uint32_t ruse = chunk_seq >> 1;
                    if (ruse > 0 && !mbar_wait(bar(gbar_r_free(rb)), (ruse - 1) & 1, abort_flag)) { ok = false; break; }
                    mbar_arrive_expect_tx(bar(gbar_r_full(rb)), kRBytes + kBiasBytes);
                    tma_load_2d(base + GSmem::rtab + rb * kRBytes, &r_map, ch * kNC, inst * P.sumM + P.mfirst[a], bar(gbar_r_full(rb)));
                    tma_load_2d(base + GSmem::bias + rb * G::BiasSlot, &b_map, ch * kNC, d.x, bar(gbar_r_full(rb)));
                    for (int ks = 0; ks < n_ks; ++ks, ++slab_seq) {
                        const int s = slab_seq % kBStages;
                        const uint32_t use = slab_seq / kBStages;
                        if (use > 0 && !mbar_wait(bar(gbar_free_b(s)), (use - 1) & 1, abort_flag)) { ok = false; break; }
                        mbar_arrive_expect_tx(bar(gbar_full_b(s)), kBSlabBytes);
                        const uint32_t bdst = base + GSmem::b_ring + s * G::BSlot;
                        tma_load_2d(bdst, &wt_map, ks * kKSlab, wrow0 + ch * kNC, bar(gbar_full_b(s)));
                        if (F32) tma_load_2d(bdst + kNC * 128, &wt_map, ks * kKSlab, prm.lo_row0 + wrow0 + ch * kNC, bar(gbar_full_b(s)));
                    }
                }
            }
        }
    } else if (warp == kGMmaWarp) {
        // ================================================================ MMA issuer (one thread)
        if (lane == 0) {
            uint32_t slab_seq = 0, chunk_seq = 0;
            bool ok = true;
            for (int it = blockIdx.x; it < n_items && ok; it += gridDim.x) {
                const int t = it / S, hf = it - t * S;
                const int4 d = prm.tiles[t];
                if (d.x < 0) continue;
                for (int ch = hf * n_ch / S; ch < (hf + 1) * n_ch / S && ok; ++ch, ++chunk_seq) {
                    const uint32_t b = chunk_seq & 1, acc_use = chunk_seq >> 1;
                    if (acc_use > 0 && !mbar_wait(bar(gbar_acc_empty(b)), (acc_use - 1) & 1, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const int ncols = min(kNC, ((C - ch * kNC) + 15) & ~15);
                    const uint32_t idesc = F32 ? instr_desc(ncols) : instr_desc_bf16(ncols);
                    const uint32_t d_tmem = b * kNC;
                    for (int ks = 0; ks < n_ks; ++ks, ++slab_seq) {
                        const int s = slab_seq % kAStages, sb = slab_seq % kBStages;
                        if (!mbar_wait(bar(gbar_full_a(s)), (slab_seq / kAStages) & 1, abort_flag)) { ok = false; break; }
                        if (!mbar_wait(bar(gbar_full_b(sb)), (slab_seq / kBStages) & 1, abort_flag)) { ok = false; break; }
                        tc_fence_after();
                        const uint64_t a_desc = smem_desc(base + GSmem::a_ring + s * kASlabBytes);
                        const uint64_t b_desc = smem_desc(base + GSmem::b_ring + sb * G::BSlot);
                        if (F32) {
                            const uint64_t bl_desc = b_desc + (uint64_t)((kNC * 128) >> 4);      // W_lo rows
                            const uint32_t a_lo = (uint32_t)(G::TmemLo + s * 32);                  // x_lo of this stage
#pragma unroll
                            for (int k = 0; k < kKSlab / 8; ++k) {
                                umma_tf32(d_tmem, a_desc + (uint64_t)(k * 2), b_desc + (uint64_t)(k * 2), idesc, (ks | k) != 0);
                                umma_tf32(d_tmem, a_desc + (uint64_t)(k * 2), bl_desc + (uint64_t)(k * 2), idesc, 1u);
                                umma_tf32_ts(d_tmem, a_lo + k * 8, b_desc + (uint64_t)(k * 2), idesc, 1u);
                            }
                        } else {
#pragma unroll
                            for (int k = 0; k < kKSlab / 16; ++k)
                                umma_bf16(d_tmem, a_desc + (uint64_t)(k * 2), b_desc + (uint64_t)(k * 2), idesc, (ks | k) != 0);
                        }
                        umma_commit(bar(gbar_free_a(s)));
                        umma_commit(bar(gbar_free_b(sb)));
                    }
                    if (ok) umma_commit(bar(gbar_acc_full(b)));
                }
            }
            if (*abort_flag) {                                 // leaving early: let the issued MMAs finish first
                umma_commit(bar(kGBarDrain));
                const unsigned long long t0 = global_ns();
                while (!mbar_try_wait(bar(kGBarDrain), 0) && global_ns() - t0 < kWaitLimitNs) {}
            }
        }
    } else if (warp < kGEpiWarp0) {
        // ================================================================ A producers: gather the rows of the tile
        const int aquad = warp & 3, row = aquad * 32 + lane;  // fp32: the thread's row is also its tensor-memory lane
        const int pt = (warp - kGAWarp0) * 32 + lane;          // copies: piece pt & 7 of rows (pt >> 3) + 16 i, i = 0..7
        const int pj = pt & 7, pr0 = pt >> 3;
        constexpr int kEsz = F32 ? 4 : 2, kPiece = 16 / kEsz; // bytes per feature, features per 16-byte piece
        uint32_t slab_seq = 0;
        bool ok = true;
        uint32_t issued = 0, signalled = 0;                    // slabs whose copies were issued / reported complete
        // This thread's copies of stage ps have landed.  fp32: once every producer's have (the row a thread reads was
        // copied by eight others), store the row's x_lo into the stage's tensor-memory slot.  Then tell the MMA issuer
        // that the A operand of the stage is complete.
        auto signal = [&](int ps, uint32_t use) -> bool {
            if (F32) {
                mbar_arrive(bar(gbar_landed(ps)));
                if (!warp_wait(bar(gbar_landed(ps)), use & 1, abort_flag)) return false;
                const unsigned char *xrow = sm + GSmem::a_ring + ps * kASlabBytes + row * 128;
                uint32_t v[32];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const uint4 q = *reinterpret_cast<const uint4 *>(xrow + ((j ^ (row & 7)) << 4));
                    v[4 * j] = q.x; v[4 * j + 1] = q.y; v[4 * j + 2] = q.z; v[4 * j + 3] = q.w;
                }
#pragma unroll
                for (int k = 0; k < 32; ++k) {
                    const float x = __uint_as_float(v[k]);
                    v[k] = __float_as_uint(x - tf32_part(x));
                }
                tc_fence_after();
                tmem_st32(((uint32_t)(aquad * 32) << 16) + (uint32_t)(G::TmemLo + ps * 32), v);
                tmem_wait_st();
                tc_fence_before();
            }
            fence_proxy_async();
            mbar_arrive(bar(gbar_full_a(ps)));
            return true;
        };
        for (int it = blockIdx.x; it < n_items && ok; it += gridDim.x) {
            const int t = it / S, hf = it - t * S;
            const int4 d = prm.tiles[t];
            if (d.x < 0) continue;
            const unsigned char *srcs[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int r = pr0 + 16 * i;
                srcs[i] = (const unsigned char *)tb.feats + tb.perm[d.y + (r < d.z ? r : 0)] * D * kEsz;
            }
            for (int ch = hf * n_ch / S; ch < (hf + 1) * n_ch / S && ok; ++ch) {
                for (int ks = 0; ks < n_ks; ++ks, ++slab_seq) {
                    const int s = slab_seq % kAStages;
                    const uint32_t use = slab_seq / kAStages;
                    if (use > 0 && !warp_wait(bar(gbar_free_a(s)), (use - 1) & 1, abort_flag)) { ok = false; break; }
                    const int kk = ks * kKSlab + pj * kPiece;
                    const int left = (D - kk) * kEsz;          // bytes of a row that exist from this piece on
                    const uint32_t nbytes = left >= 16 ? 16u : left > 0 ? (uint32_t)left : 0u;
                    const int koff = (kk < D ? kk : 0) * kEsz;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const int r = pr0 + 16 * i;
                        cp_async16_zfill(base + GSmem::a_ring + s * kASlabBytes + r * 128 + ((pj ^ (r & 7)) << 4), srcs[i] + koff, nbytes);
                    }
                    cp_async_commit();
                    ++issued;
                    if (issued - signalled > (uint32_t)G::ADepth) {    // keep ADepth slabs in flight: the oldest has landed
                        cp_async_wait<G::ADepth>();
                        if (!signal((int)(signalled % kAStages), signalled / kAStages)) { ok = false; break; }
                        ++signalled;
                    }
                }
            }
        }
        cp_async_wait<0>();
        while (ok && signalled < issued) {
            if (!signal((int)(signalled % kAStages), signalled / kAStages)) break;
            ++signalled;
        }
    } else {
        // ================================================================ epilogue warps (one row per thread, a quarter of the columns)
        const int eg = (warp - kGEpiWarp0) >> 2;               // column group of every chunk this warpgroup reads
        const int quad = warp & 3, row = quad * 32 + lane;
        const float *rtab = reinterpret_cast<const float *>(sm + GSmem::rtab);
        const float *btab = reinterpret_cast<const float *>(sm + GSmem::bias);
        float *merge_all = reinterpret_cast<float *>(sm + GSmem::merge);
        uint32_t chunk_seq = 0, tile_seq = 0;
        const int Mmax = P.Mmax;
        bool ok = true;
        constexpr int kGW = kNC / kGEpiGroups;                     // columns of a chunk per epilogue group
        constexpr int kBlk = kGEpiBlk;
        constexpr float kMScale = F32 ? 1.f : kLog2e;                // units of the running maximum: base-2 (fp32) or natural (bf16) logits
        static_assert(kNC % (4 * kGEpiGroups) == 0, "a group's first column must keep 16-byte alignment in the tables");
        for (int it = blockIdx.x; it < n_items && ok; it += gridDim.x) {
            const int t = it / S, hf = it - t * S;
            const int4 d = prm.tiles[t];
            if (d.x < 0) continue;
            const int inst = d.x / A, a = d.x - inst * A;
            const int g0 = P.mfirst[a], M = P.mfirst[a + 1] - g0;
            float run_m = -INFINITY, run_s = 0.f, racc[kMaxModelsPerApp];
#pragma unroll
            for (int j = 0; j < kMaxModelsPerApp; ++j) racc[j] = 0.f;
            for (int ch = hf * n_ch / S; ch < (hf + 1) * n_ch / S && ok; ++ch, ++chunk_seq) {
                const uint32_t b = chunk_seq & 1, par = (chunk_seq >> 1) & 1;
                if (!warp_wait(bar(gbar_r_full(b)), par, abort_flag)) { ok = false; break; }
                if (!warp_wait(bar(gbar_acc_full(b)), par, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const float *rt = rtab + b * (kRBytes / 4), *bt = btab + b * (G::BiasSlot / 4);
                const int c_base = ch * kNC;
                for (int sb = 0; sb < (kGW + kBlk - 1) / kBlk; ++sb) {
                    const int col0 = eg * kGW + sb * kBlk;                 // column of the chunk
                    const int col_end = (eg + 1) * kGW;                    // this group's columns end here
                    if (c_base + col0 >= C) break;                         // uniform: nothing valid from here on
                    float z[kBlk];
                    tmem_ld<kBlk>(((uint32_t)(quad * 32) << 16) + b * kNC + col0, z);
                    tmem_wait_ld();
                    float bm = -INFINITY;
#pragma unroll
                    for (int c = 0; c < kBlk; c += 4) {
                        if (col0 + c < kNC) {                              // the bias row has NC entries
                            const float4 bv = *reinterpret_cast<const float4 *>(bt + col0 + c);
                            if (F32) {                                     // log2(e) is already in the head image
                                z[c] = fmaf(bv.x, kLog2e, z[c]); z[c + 1] = fmaf(bv.y, kLog2e, z[c + 1]);
                                z[c + 2] = fmaf(bv.z, kLog2e, z[c + 2]); z[c + 3] = fmaf(bv.w, kLog2e, z[c + 3]);
                            } else {
                                z[c] += bv.x; z[c + 1] += bv.y; z[c + 2] += bv.z; z[c + 3] += bv.w;   // natural units; log2(e) goes into the exponent's FMA
                            }
                        }
                    }
                    if (c_base + col0 + kBlk <= C && col0 + kBlk <= col_end) {   // whole block valid (uniform): no masking
#pragma unroll
                        for (int c = 0; c < kBlk; ++c) bm = fmaxf(bm, z[c]);
                    } else {
#pragma unroll
                        for (int c = 0; c < kBlk; ++c) {
                            if (c_base + col0 + c >= C || col0 + c >= col_end) z[c] = -INFINITY;
                            bm = fmaxf(bm, z[c]);
                        }
                    }
                    if (bm > run_m) {                                      // rescale what has been summed so far
                        const float sc = exp2_unit((run_m - bm) * kMScale); // 0 for the first block (run_m = -inf)
                        run_s *= sc;
#pragma unroll
                        for (int j = 0; j < kMaxModelsPerApp; ++j) racc[j] *= sc;
                        run_m = bm;
                    }
                    float ps = 0.f;
                    if (F32) {
#pragma unroll
                        for (int c = 0; c < kBlk; ++c) { z[c] = exp2_unit(z[c] - run_m); ps += z[c]; }
                    } else {
                        const float nm = -run_m * kLog2e;
#pragma unroll
                        for (int c = 0; c < kBlk; ++c) { z[c] = exp2_unit(fmaf(z[c], kLog2e, nm)); ps += z[c]; }
                    }
                    run_s += ps;
                    // recall contraction with two-wide FMAs: label pairs (c, c + 1) of a model's row against the pair of
                    // numerators; the two halves of the accumulator are added once per block of labels
                    unsigned long long zz[kBlk / 2];
#pragma unroll
                    for (int c = 0; c < kBlk / 2; ++c) zz[c] = pack_f32x2(z[2 * c], z[2 * c + 1]);
#pragma unroll
                    for (int j = 0; j < kMaxModelsPerApp; j += 2) {        // two models at a time: four independent chains
                        if (j < M) {
                            const float *r0 = rt + j * kNC + col0, *r1 = j + 1 < M ? r0 + kNC : r0;
                            unsigned long long p0a = 0ull, p0b = 0ull, p1a = 0ull, p1b = 0ull;
#pragma unroll
                            for (int c = 0; c < kBlk; c += 4) {
                                if (col0 + c < kNC) {                      // a recall row has NC entries; z is 0 past the group's end
                                    const ulonglong2 rv0 = *reinterpret_cast<const ulonglong2 *>(r0 + c);
                                    const ulonglong2 rv1 = *reinterpret_cast<const ulonglong2 *>(r1 + c);
                                    fma_f32x2(p0a, zz[c >> 1], rv0.x);
                                    fma_f32x2(p1a, zz[c >> 1], rv1.x);
                                    fma_f32x2(p0b, zz[(c >> 1) + 1], rv0.y);
                                    fma_f32x2(p1b, zz[(c >> 1) + 1], rv1.y);
                                }
                            }
                            racc[j] += sum_f32x2(p0a) + sum_f32x2(p0b);
                            if (j + 1 < M) racc[j + 1] += sum_f32x2(p1a) + sum_f32x2(p1b);
                        }
                    }
                }
                tc_fence_before();
                mbar_arrive(bar(gbar_acc_empty(b)));
                mbar_arrive(bar(gbar_r_free(b)));
            }
            if (!ok) break;
            // ---- merge the column groups of the row, finish Eq. 9 / Eq. 12, store
            if (eg > 0) {
                float *merge = merge_all + ((eg - 1) * kGRows + row) * kMergeFloats;
                if (tile_seq > 0 && !warp_wait(bar(kGBarMergeDone), (tile_seq - 1) & 1, abort_flag)) break;
                merge[0] = run_m; merge[1] = run_s;
#pragma unroll
                for (int j = 0; j < kMaxModelsPerApp; ++j) merge[2 + j] = racc[j];
                mbar_arrive(bar(kGBarMergeReady));
            } else {
                if (!warp_wait(bar(kGBarMergeReady), tile_seq & 1, abort_flag)) break;
                float mm = run_m;
#pragma unroll
                for (int g = 0; g < kGEpiGroups - 1; ++g) mm = fmaxf(mm, merge_all[(g * kGRows + row) * kMergeFloats]);
                const float s0 = run_m == -INFINITY ? 0.f : exp2_unit((run_m - mm) * kMScale);
                float tot = run_s * s0;
#pragma unroll
                for (int j = 0; j < kMaxModelsPerApp; ++j) racc[j] *= s0;
#pragma unroll
                for (int g = 0; g < kGEpiGroups - 1; ++g) {
                    const float *mg = merge_all + (g * kGRows + row) * kMergeFloats;
                    const float om = mg[0];
                    const float sg = om == -INFINITY ? 0.f : exp2_unit((om - mm) * kMScale);
                    tot = fmaf(mg[1], sg, tot);
#pragma unroll
                    for (int j = 0; j < kMaxModelsPerApp; ++j) racc[j] = fmaf(mg[2 + j], sg, racc[j]);
                }
                bool last = true;
                if (S > 1) {
                    // this half's state of the row goes to global memory; the half that arrives second finds the other
                    // one's there (fence before the counter on both sides) and finishes the row
                    float *mine = prm.partial + ((size_t)(t * 2 + hf) * kMergeFloats) * kGRows + row;
                    mine[0] = mm; mine[kGRows] = tot;
#pragma unroll
                    for (int j = 0; j < kMaxModelsPerApp; ++j) mine[(2 + j) * kGRows] = racc[j];
                    __threadfence();
                    last = atomicAdd(prm.part_count + (size_t)t * kGRows + row, 1) == 1;
                    if (last) {
                        __threadfence();
                        const float *other = prm.partial + ((size_t)(t * 2 + (1 - hf)) * kMergeFloats) * kGRows + row;
                        const float om = __ldcg(other), os = __ldcg(other + kGRows);
                        const float m2 = fmaxf(mm, om);
                        const float sa = mm == -INFINITY ? 0.f : exp2_unit((mm - m2) * kMScale);
                        const float sb = om == -INFINITY ? 0.f : exp2_unit((om - m2) * kMScale);
                        tot = fmaf(os, sb, tot * sa);
#pragma unroll
                        for (int j = 0; j < kMaxModelsPerApp; ++j) racc[j] = fmaf(__ldcg(other + (2 + j) * kGRows), sb, racc[j] * sa);
                    }
                }
                const float inv = 1.f / tot;
                const bool valid = last && row < d.z;
                const int64_t req = tb.perm[d.y + (valid ? row : 0)];
                float *dst = tb.acc32 + req * Mmax;
                float *dst2 = prm.acc_out ? prm.acc_out + req * Mmax : nullptr;
                float a0 = 0.f, q1 = 0.f, q2 = 0.f;
#pragma unroll
                for (int j = 0; j < kMaxModelsPerApp; ++j) {
                    if (j < Mmax) {
                        float aj = 0.f;
                        if (j < M) {
                            aj = racc[j] * inv;
                            if (P.prior)
                                aj = (P.prior_dot[(int64_t)inst * P.sumM + g0 + j] + P.kappa * aj) / (P.prior_sum[d.x] + P.kappa);
                            if (j == 0) a0 = aj;
                            const float dj = aj - a0;
                            q1 += dj; q2 = fmaf(dj, dj, q2);
                        }
                        if (valid) {
                            dst[j] = aj;
                            if (dst2) dst2[j] = aj;
                        }
                    }
                }
                if (valid) {
                    const float invM = 1.f / (float)M, md = q1 * invM;
                    tb.v32[req] = 1.f + fmaxf(fmaf(q2, invM, -md * md), 0.f);
                }
                mbar_arrive(bar(kGBarMergeDone));
            }
            ++tile_seq;
        }
    }

    // ---- teardown
    tc_fence_before();
    __syncthreads();
    if (tid == 0 && *abort_flag) dev_error(&prm.flags[0], kDevLimit);
    if (warp == kGMmaWarp) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512) : "memory");
    }
}

}  // namespace gemm
}  // namespace sp
