// Tensor-core scoring kernel for small heads (fp32 features, D <= 128, all applications' labels fit
// in 64 logit columns).  Persistent, warp-specialised, one thread block per SM.
//
// Per request (Section 4.1 + Eq. 9 + Eq. 12 of the paper):
//   z = x W_a + b_a;  p = softmax(z);  theta = Dirichlet posterior mean;  acc_j = sum_c theta_c recall_j(c);
//   v = 1 + population variance_j(acc_j).
// The step is bound by reading x from HBM once; at ~10 flop per byte the FP32 pipes cannot keep up with
// HBM3e, so the logits are computed by the tcgen05 tensor cores:
//   * a tile is 128 consecutive requests of one instance; TMA brings it into shared memory as K-major,
//     128-byte-swizzled slabs of 128 rows x 32 features (the layout the MMA reads directly);
//   * the logits of ALL applications of the instance are computed for every row ([A*C] <= 64 columns);
//     each row later keeps the columns of its own application, so rows need no regrouping;
//   * fp32 accuracy from the tf32 unit: x = x_hi + x_lo and W = W_hi + W_lo with x_hi, W_hi the values
//     truncated to tf32 (what the unit reads from a 32-bit container) and the remainders exact in fp32;
//     z = x_hi W_hi + x_hi W_lo + x_lo W_hi accumulates in fp32 in tensor memory, the dropped x_lo W_lo term
//     is below 2^-20 relative;
//   * shared-memory bandwidth is the scarce resource (every MMA re-reads its operands), so the A operand
//     comes from tensor memory: converter warps (one row per thread) read each slab once, store the row as
//     loaded (read as x_hi) and its remainder x_lo into a ring of tensor-memory columns, and the MMAs read
//     only the small W operand from shared memory.  The converters also rebuild the W operand when the
//     instance changes;
//   * epilogue warps read the accumulator from tensor memory (one row per thread), add the bias, and do
//     softmax, the recall contraction, the Dirichlet step and the variance in registers.
// Every wait on an mbarrier is bounded; when a wait runs out the block raises kDevLimit and leaves.
#pragma once

#include <cuda.h>

#include "sp_common.cuh"
#include "sp_group.cuh"

namespace sp {
namespace mma {

constexpr int kRows = 128;                 // requests per tile = MMA M
constexpr int kSlabK = 32;                 // features per slab row (128 bytes)
constexpr int kSlabBytes = kRows * 128;    // 16 KB: 128 rows x 128 bytes
constexpr int kMaxD = 128;
constexpr int kMaxSlabs = kMaxD / kSlabK;
constexpr int kCols = 64;                  // logit columns (sum over applications of the label count)
constexpr int kXStages = 6;                // ring of slabs in shared memory filled by TMA
constexpr int kASlots = 6;                 // ring of A operands in tensor memory: 32 columns x_hi + 32 columns x_lo each
constexpr int kTmemCols = 512;             // whole tensor memory
constexpr int kAccCols = 64;               // columns per accumulator: x_hi W_hi + x_hi W_lo + x_lo W_hi, all applications
constexpr int kTmemA = 2 * kAccCols;       // accumulators first (epilogue reads may overhang into the A ring), then the ring
constexpr int kSlotCols = 2 * kSlabK;
constexpr int kProducerWarp = 0, kMmaWarp = 1, kConvWarp0 = 2, kEpiWarp0 = 6;
constexpr int kEpiGroups = 2;              // epilogue warpgroups; group g takes every second tile and accumulator g
constexpr int kMmaWarp2 = 6 + 4 * kEpiGroups;   // second MMA issuer: the two take alternate tiles (and accumulators)
constexpr int kThreads = 32 * (7 + 4 * kEpiGroups);
constexpr int kConvThreads = 128, kEpiThreads = 128;
constexpr float kLog2e = 1.44269502162933349609375f;   // folded into W and the bias: the softmax runs in base 2
constexpr int kWChunks = (kCols * kMaxD / 4) / kConvThreads;  // 4-feature pieces of the head operand per converter thread
constexpr unsigned long long kWaitLimitNs = 1000ull * 1000ull * 1000ull;

struct Smem {                               // byte offsets from the 1024-byte aligned base
    static constexpr int w = 0;                                        // kMaxSlabs slabs: rows 0..63 W_hi, 64..127 W_lo
    static constexpr int wraw = w + kMaxSlabs * kSlabBytes;            // the next instance's heads as stored: W[a][d][c] fp32
    static constexpr int x = wraw + kCols * kMaxD * 4;
    // per-instance tables, one copy per epilogue group, label rows padded with zeros to a multiple of 4 floats (Cp):
    // recall [sumM][Cp] (<= 1024 floats), bias * log2(e) [A][Cp] (<= 128), prior_dot [sumM] (<= 256), prior_sum [A] (<= 16)
    static constexpr int tab_recall = 0, tab_bias = 1024, tab_pdot = tab_bias + 2 * kCols, tab_psum = tab_pdot + 256;
    static constexpr int tab_floats = tab_psum + 16;
    static constexpr int tabs = x + kXStages * kSlabBytes;
    static constexpr int bars = tabs + kEpiGroups * tab_floats * 4;
    static constexpr int n_bars = 2 * kXStages + 3 * kASlots + 9 + 2 * kEpiGroups;
    static constexpr int misc = bars + n_bars * 8;                     // tmem base, abort flag
    static constexpr int end = misc + 16;
    static constexpr int bytes = end + 1024;                           // slack for the manual alignment
};

struct Params {
    DevProfiles P;
    DevTable tb;
    const int4 *tiles;       // (instance, first request relative to the instance, rows, first request in the table)
    int n_tiles;             // entries in `tiles`; the valid ones come first, those past the end have instance -1
    float *acc_out;          // optional second destination of acc
    int *flags;
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n.reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait: false when the wait ran out (the block-wide abort flag is then set) or another thread gave up.
// The polling loop is kept out of line: it is entered only when the barrier is not ready yet.
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int *abort_flag) {
    const unsigned long long t0 = global_ns();
    for (uint32_t it = 1;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 63) == 0) {
            if (*abort_flag) return false;
            if (global_ns() - t0 > kWaitLimitNs) { *abort_flag = 1; return false; }
            __nanosleep(64);
        }
    }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag) {
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, abort_flag);
}

__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// 2-D tiled TMA load (no multicast): box of the tensor map at (x = feature, y = request) -> shared memory.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
        : "memory");
}

// Plain bulk copy global -> shared memory (no multicast); both addresses and the size are multiples of 16 bytes.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
    uint64_t d = (uint64_t)((addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)1 << 16;              // leading byte offset (not used by swizzled K-major layouts)
    d |= (uint64_t)(1024 >> 4) << 32;    // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;              // descriptor version of this architecture
    d |= (uint64_t)2 << 61;              // 128-byte swizzle
    return d;
}
// Instruction descriptor: tf32 x tf32 -> fp32, both operands K-major, M = 128, N = n.
__host__ __device__ constexpr uint32_t instr_desc(int n) {
    return (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kRows >> 4) << 24);
}
__device__ __forceinline__ void umma_tf32(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n.reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc)
        : "memory");
}
// Same with the A operand in tensor memory (128 lanes x 8 columns of 32-bit containers per instruction).
__device__ __forceinline__ void umma_tf32_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n.reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %2, %3, p;\n}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(acc)
        : "memory");
}
// Arrives on the mbarrier once every MMA issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

template <int N>
__device__ __forceinline__ void tmem_ld(uint32_t taddr, float (&r)[N]);
template <>
__device__ __forceinline__ void tmem_ld<16>(uint32_t taddr, float (&r)[16]) {
    uint32_t v[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr)
        : "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) r[i] = __uint_as_float(v[i]);
}
template <>
__device__ __forceinline__ void tmem_ld<32>(uint32_t taddr, float (&r)[32]) {
    uint32_t v[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
          "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
          "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) r[i] = __uint_as_float(v[i]);
}
template <>
__device__ __forceinline__ void tmem_ld<8>(uint32_t taddr, float (&r)[8]) {
    uint32_t v[8];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
                 : "r"(taddr)
                 : "memory");
#pragma unroll
    for (int i = 0; i < 8; ++i) r[i] = __uint_as_float(v[i]);
}
template <>
__device__ __forceinline__ void tmem_ld<24>(uint32_t taddr, float (&r)[24]) {
    float a[16], b[8];
    tmem_ld<16>(taddr, a);
    tmem_ld<8>(taddr + 16, b);
#pragma unroll
    for (int i = 0; i < 16; ++i) r[i] = a[i];
#pragma unroll
    for (int i = 0; i < 8; ++i) r[16 + i] = b[i];
}
template <>
__device__ __forceinline__ void tmem_ld<48>(uint32_t taddr, float (&r)[48]) {
    float a[32], b[16];
    tmem_ld<32>(taddr, a);
    tmem_ld<16>(taddr + 32, b);
#pragma unroll
    for (int i = 0; i < 32; ++i) r[i] = a[i];
#pragma unroll
    for (int i = 0; i < 16; ++i) r[32 + i] = b[i];
}
template <>
__device__ __forceinline__ void tmem_ld<64>(uint32_t taddr, float (&r)[64]) {
    float a[32], b[32];
    tmem_ld<32>(taddr, a);
    tmem_ld<32>(taddr + 32, b);
#pragma unroll
    for (int i = 0; i < 32; ++i) { r[i] = a[i]; r[32 + i] = b[i]; }
}
// 32 consecutive columns of this thread's lane.
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
        "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
        ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]),
          "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]), "r"(v[16]), "r"(v[17]),
          "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]), "r"(v[24]), "r"(v[25]), "r"(v[26]),
          "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31])
        : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Value a tf32 operand takes from a 32-bit container: the low 13 mantissa bits are not read.
__device__ __forceinline__ float tf32_part(float x) { return __uint_as_float(__float_as_uint(x) & 0xFFFFE000u); }

// 2^x from the ex2 unit (about 2^-22 relative error; 2^-inf = 0).
__device__ __forceinline__ float exp2_unit(float x) {
    float p;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(p) : "f"(x));
    return p;
}

// Barrier indices
constexpr int kBarBase2 = 2 * kXStages + 3 * kASlots;
__device__ __forceinline__ constexpr int bar_full(int h) { return h; }                       // slab landed in shared memory
__device__ __forceinline__ constexpr int bar_x_free(int h) { return kXStages + h; }          // converters are done with the slab
// A operand slot l written for MMA issuer g (each issuer waits on its own barriers: a waiter that is a whole
// phase ahead of another one would pass a shared barrier early)
__device__ __forceinline__ constexpr int bar_a_ready(int g, int l) { return 2 * kXStages + g * kASlots + l; }
__device__ __forceinline__ constexpr int bar_a_free(int l) { return 2 * kXStages + 2 * kASlots + l; }   // its MMAs completed
__device__ __forceinline__ constexpr int bar_acc_full(int b) { return kBarBase2 + b; }
__device__ __forceinline__ constexpr int bar_acc_empty(int b) { return kBarBase2 + 2 + b; }
constexpr int kBarDrain = kBarBase2 + 5;
constexpr int kBarRawFull = kBarBase2 + 6;    // raw heads of an instance landed in shared memory
constexpr int kBarRawFree = kBarBase2 + 7;    // converters have turned them into the operand
constexpr int kBarDrain2 = kBarBase2 + 8;     // drain barrier of the second MMA issuer
// per epilogue group: A = every thread is done reading the old tables, B = the new tables are written
__device__ __forceinline__ constexpr int bar_epi_a(int g) { return kBarBase2 + 9 + g; }
__device__ __forceinline__ constexpr int bar_epi_b(int g) { return kBarBase2 + 9 + kEpiGroups + g; }

// Warp-uniform outcome of a bounded wait done by every lane.
__device__ __forceinline__ bool warp_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag) {
    const bool ok = mbar_wait(bar, parity, abort_flag);
    return __all_sync(0xffffffffu, ok);
}

// CT = logit columns one epilogue thread keeps in registers (>= C); PRIOR = a Dirichlet prior is set (without it the
// code of that step is left out).
template <int CT, bool PRIOR>
__global__ void __launch_bounds__(kThreads, 1)
k_score_mma(const __grid_constant__ CUtensorMap x_map, const Params prm) {
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw_u32 = smem_u32(smem_raw);
    const uint32_t base = (raw_u32 + 1023u) & ~1023u;
    unsigned char *sm = smem_raw + (base - raw_u32);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(sm + Smem::misc);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(sm + Smem::misc + 4);
    auto bar = [&](int i) -> uint32_t { return base + Smem::bars + 8u * (uint32_t)i; };

    const DevProfiles &P = prm.P;
    const DevTable &tb = prm.tb;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int A = P.A, C = P.C, D = P.D;
    const int n_slabs = (D + kSlabK - 1) / kSlabK;
    const int per_cta = (prm.n_tiles + (int)gridDim.x - 1) / (int)gridDim.x;
    const int t_begin = (int)blockIdx.x * per_cta;
    const int t_end = min(t_begin + per_cta, prm.n_tiles);

    // ---- set-up: barriers, tensor memory, zeroed W operand (padding rows and features stay zero)
    if (tid == 0) {
        for (int h = 0; h < kXStages; ++h) { mbar_init(bar(bar_full(h)), 1); mbar_init(bar(bar_x_free(h)), kConvThreads); }
        for (int l = 0; l < kASlots; ++l) {
            mbar_init(bar(bar_a_ready(0, l)), kConvThreads); mbar_init(bar(bar_a_ready(1, l)), kConvThreads);
            mbar_init(bar(bar_a_free(l)), 1);
        }
        for (int b = 0; b < 2; ++b) { mbar_init(bar(bar_acc_full(b)), 1); mbar_init(bar(bar_acc_empty(b)), kEpiThreads); }
        mbar_init(bar(kBarDrain), 1);
        mbar_init(bar(kBarDrain2), 1);
        mbar_init(bar(kBarRawFull), 1);
        mbar_init(bar(kBarRawFree), kConvThreads);
        for (int g = 0; g < kEpiGroups; ++g) { mbar_init(bar(bar_epi_a(g)), kEpiThreads); mbar_init(bar(bar_epi_b(g)), kEpiThreads); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int k = tid; k < kMaxSlabs * kSlabBytes / 16; k += kThreads)
        reinterpret_cast<float4 *>(sm + Smem::w)[k] = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int k = tid; k < kEpiGroups * Smem::tab_floats; k += kThreads)      // the padding of the label rows stays zero
        reinterpret_cast<float *>(sm + Smem::tabs)[k] = 0.f;
    if (warp == kMmaWarp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    if (tmem != 0 && tid == 0) *abort_flag = 1;                // cannot happen for a whole-memory allocation
    __syncthreads();
    const bool tmem_ok = *abort_flag == 0;

    if (!tmem_ok) {
        // unexpected tensor-memory base: nothing runs, the block reports the error below
    } else if (warp == kProducerWarp) {
        // ================================================================ TMA producer (one thread)
        if (lane == 0) {
            uint32_t slab_seq = 0, w_seq = 0;
            int cur_inst = -1;
            const uint32_t w_bytes = (uint32_t)(A * D * C) * 4u;
            bool ok = true;
            int4 d_next = t_begin < t_end ? prm.tiles[t_begin] : make_int4(-1, 0, 0, 0);
            for (int t = t_begin; t < t_end && ok; ++t) {
                const int4 d = d_next;
                if (d.x < 0) break;                            // valid tiles form a prefix of the block's range
                if (t + 1 < t_end) d_next = prm.tiles[t + 1];
                if (d.x != cur_inst) {                         // stage the heads of the instance this tile starts
                    if (w_seq > 0 && !mbar_wait(bar(kBarRawFree), (w_seq - 1) & 1, abort_flag)) break;
                    mbar_arrive_expect_tx(bar(kBarRawFull), w_bytes);
                    bulk_load(base + Smem::wraw, (const float *)P.W + (int64_t)d.x * A * D * C, w_bytes, bar(kBarRawFull));
                    ++w_seq; cur_inst = d.x;
                }
                const int row0 = d.w;
                for (int s = 0; s < n_slabs; ++s, ++slab_seq) {
                    const int h = slab_seq % kXStages;
                    const uint32_t use = slab_seq / kXStages;
                    if (use > 0 && !mbar_wait(bar(bar_x_free(h)), (use - 1) & 1, abort_flag)) { ok = false; break; }
                    mbar_arrive_expect_tx(bar(bar_full(h)), kSlabBytes);
                    tma_load_2d(base + Smem::x + h * kSlabBytes, &x_map, s * kSlabK, row0, bar(bar_full(h)));
                }
            }
            if (!ok || *abort_flag) {
                // copies already issued still land in shared memory: give them a bounded time to finish
                if (w_seq > 0) {
                    const unsigned long long t0 = global_ns();
                    while (!mbar_try_wait(bar(kBarRawFull), (w_seq - 1) & 1) && global_ns() - t0 < kWaitLimitNs) {}
                }
                const uint32_t first = slab_seq > (uint32_t)kXStages ? slab_seq - kXStages : 0;
                for (uint32_t q = first; q < slab_seq; ++q) {
                    const unsigned long long t0 = global_ns();
                    while (!mbar_try_wait(bar(bar_full(q % kXStages)), (q / kXStages) & 1) && global_ns() - t0 < kWaitLimitNs) {}
                }
            }
        }
    } else if (warp == kMmaWarp || warp == kMmaWarp2) {
        // ================================================================ MMA issuers (one thread each)
        // Issuing an MMA costs about as much time as the tensor pipe needs for it at this tile shape, so two
        // threads issue: issuer g takes tiles g, g + 2, ... and accumulator g; their MMAs interleave in the pipe.
        // All tensor-memory addresses below are compile-time offsets: the allocation covers the whole tensor
        // memory, so its base is column 0 (checked after the allocation).
        if (lane == 0) {
            constexpr uint32_t idesc = instr_desc(kCols);
            constexpr uint64_t w_lo_rows = (uint64_t)((kCols * 128) >> 4);   // operand rows 64..127 hold W_lo
            const uint64_t w_desc = smem_desc(base + Smem::w);
            const int mg = warp == kMmaWarp ? 0 : 1;
            bool ok = true;
            uint32_t rdy_par = 0;                              // bit l: parity of this issuer's next wait on slot l
            int4 d_next = t_begin + mg < t_end ? prm.tiles[t_begin + mg] : make_int4(-1, 0, 0, 0);
            for (int t = t_begin + mg; t < t_end && ok; t += 2) {
                const int4 d = d_next;
                if (d.x < 0) break;                            // valid tiles form a prefix of the block's range
                if (t + 2 < t_end) d_next = prm.tiles[t + 2];
                const uint32_t tile_seq = (uint32_t)(t - t_begin);
                uint32_t slab_seq = tile_seq * (uint32_t)n_slabs;
                const uint32_t b = tile_seq & 1, acc_use = tile_seq >> 1;
                if (acc_use > 0 && !mbar_wait(bar(bar_acc_empty(b)), (acc_use - 1) & 1, abort_flag)) break;
                tc_fence_after();
                const uint32_t d_tmem = b * kAccCols;
                for (int s = 0; s < n_slabs; ++s, ++slab_seq) {
                    const uint32_t l = slab_seq % kASlots;
                    // the slot holds the rows of this slab; the same arrival says that the head operand of the
                    // slab's features is in place (the converters rebuild it before they arrive)
                    if (!mbar_wait(bar(bar_a_ready(mg, l)), (rdy_par >> l) & 1, abort_flag)) { ok = false; break; }
                    rdy_par ^= 1u << l;
                    tc_fence_after();
                    const uint32_t a_hi = kTmemA + l * kSlotCols, a_lo = a_hi + kSlabK;
                    const uint64_t b_w = w_desc + (uint64_t)((s * kSlabBytes) >> 4);
#pragma unroll
                    for (int k = 0; k < kSlabK / 8; ++k) {     // the three products accumulate in the same 64 columns
                        umma_tf32_ts(d_tmem, a_hi + k * 8, b_w + (uint64_t)(k * 2), idesc, (s | k) != 0);
                        umma_tf32_ts(d_tmem, a_hi + k * 8, b_w + w_lo_rows + (uint64_t)(k * 2), idesc, 1u);
                        umma_tf32_ts(d_tmem, a_lo + k * 8, b_w + (uint64_t)(k * 2), idesc, 1u);
                    }
                    umma_commit(bar(bar_a_free(l)));
                }
                if (ok) umma_commit(bar(bar_acc_full(b)));
            }
            if (*abort_flag) {                                 // leaving early: let the issued MMAs finish first
                const uint32_t drain = bar(mg ? kBarDrain2 : kBarDrain);
                umma_commit(drain);
                const unsigned long long t0 = global_ns();
                while (!mbar_try_wait(drain, 0) && global_ns() - t0 < kWaitLimitNs) {}
            }
        }
    } else if (warp < kEpiWarp0) {
        // ================================================================ converter warps
        const int ct = tid - kConvWarp0 * 32;                  // 0..127
        const int cquad = warp & 3, crow = cquad * 32 + lane;  // tensor-memory lanes this warp may write = its rows
        uint32_t slab_seq = 0, w_seq = 0;
        int cur_inst = -1;
        // Head operand: this thread owns logit column wn (= operand row) and, per slab, 4 of its 8 chunks of 4
        // features.  The raw heads W[a][d][c] of the instance were staged in shared memory by the producer;
        // consecutive threads read consecutive labels (distinct banks) and write 16-byte pieces of the swizzled
        // operand rows.  The operand is rebuilt slab by slab during the first tile of an instance: slab s as soon
        // as the MMAs of the previous tile's slab s have completed, so the pipeline never drains.
        const int wn = ct & (kCols - 1), wq0 = (ct >> 6) * 4;
        const int wa = wn / C, wc = wn - wa * C;
        const bool w_row = wn < A * C;
        const float *wraw = reinterpret_cast<const float *>(sm + Smem::wraw) + wa * D * C + wc;
        bool ok = true;
        int4 d_next = t_begin < t_end ? prm.tiles[t_begin] : make_int4(-1, 0, 0, 0);
        for (int t = t_begin; t < t_end && ok; ++t) {
            const int4 d = d_next;
            if (d.x < 0) break;                                // valid tiles form a prefix of the block's range
            if (t + 1 < t_end) d_next = prm.tiles[t + 1];
            const int mg = (t - t_begin) & 1;                  // MMA issuer of this tile
            const bool new_inst = d.x != cur_inst;
            cur_inst = d.x;
            if (new_inst && !warp_wait(bar(kBarRawFull), w_seq & 1, abort_flag)) break;
            for (int s = 0; s < n_slabs; ++s, ++slab_seq) {
                const int h = slab_seq % kXStages, l = slab_seq % kASlots;
                const uint32_t a_use = slab_seq / kASlots;
                if (new_inst) {
                    // MMAs of earlier tiles on slab s read the old operand.  Slabs more than kASlots back have
                    // completed (their slots were taken again, which waited for them); the younger ones with the
                    // same s are waited for here, each on a barrier phase that cannot have been passed yet.
                    for (uint32_t back = (uint32_t)n_slabs; back <= slab_seq && back <= (uint32_t)kASlots && ok; back += (uint32_t)n_slabs) {
                        const uint32_t ps = slab_seq - back;
                        if (!warp_wait(bar(bar_a_free(ps % kASlots)), (ps / kASlots) & 1, abort_flag)) ok = false;
                    }
                    if (!ok) break;
                    if (w_row) {
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const int j = wq0 + q, dd = s * kSlabK + j * 4;   // 16-byte piece j of the operand row
                            if (dd < D) {
                                const uint32_t off = (uint32_t)(s * kSlabBytes + wn * 128 + ((j ^ (wn & 7)) << 4));
                                const float *src = wraw + dd * C;
                                const float w0 = src[0] * kLog2e, w1 = src[C] * kLog2e;
                                const float w2 = src[2 * C] * kLog2e, w3 = src[3 * C] * kLog2e;
                                float4 hi, lo;
                                hi.x = tf32_part(w0); lo.x = w0 - hi.x;
                                hi.y = tf32_part(w1); lo.y = w1 - hi.y;
                                hi.z = tf32_part(w2); lo.z = w2 - hi.z;
                                hi.w = tf32_part(w3); lo.w = w3 - hi.w;
                                *reinterpret_cast<float4 *>(sm + Smem::w + off) = hi;
                                *reinterpret_cast<float4 *>(sm + Smem::w + off + kCols * 128) = lo;
                            }
                        }
                    }
                    fence_proxy_async();
                    if (s == n_slabs - 1) { mbar_arrive(bar(kBarRawFree)); ++w_seq; }
                }
                if (!warp_wait(bar(bar_full(h)), (slab_seq / kXStages) & 1, abort_flag)) { ok = false; break; }
                // this thread's row of the slab: 8 pieces of 16 bytes, un-swizzled into feature order
                const unsigned char *xrow = sm + Smem::x + h * kSlabBytes + crow * 128;
                uint32_t v[kSlabK];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const uint4 q = *reinterpret_cast<const uint4 *>(xrow + ((j ^ (crow & 7)) << 4));
                    v[4 * j] = q.x; v[4 * j + 1] = q.y; v[4 * j + 2] = q.z; v[4 * j + 3] = q.w;
                }
                uint32_t vlo[kSlabK];                          // remainders, computed while the slot may still be busy
#pragma unroll
                for (int k = 0; k < kSlabK; ++k) {
                    const float x = __uint_as_float(v[k]);
                    vlo[k] = __float_as_uint(x - tf32_part(x));
                }
                if (a_use > 0 && !warp_wait(bar(bar_a_free(l)), (a_use - 1) & 1, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t a_hi = ((uint32_t)(cquad * 32) << 16) + (uint32_t)(kTmemA + l * kSlotCols);
                tmem_st32(a_hi, v);                            // read as x_hi: the unit drops the low mantissa bits
                tmem_st32(a_hi + kSlabK, vlo);
                tmem_wait_st();
                tc_fence_before();
                mbar_arrive(bar(bar_a_ready(mg, l)));
                mbar_arrive(bar(bar_x_free(h)));
            }
        }
    } else {
        // ================================================================ epilogue warps (one row per thread)
        const int eg = (warp - kEpiWarp0) >> 2;                // group: tiles eg, eg + 2, ... and accumulator eg
        const int et = (tid - kEpiWarp0 * 32) & (kEpiThreads - 1);
        const int quad = warp & 3;                             // tensor-memory lanes this warp may read
        const int row = quad * 32 + lane;
        float *tab = reinterpret_cast<float *>(sm + Smem::tabs) + eg * Smem::tab_floats;
        const float *recall_s = tab + Smem::tab_recall, *bias_s = tab + Smem::tab_bias;
        const float *pdot_s = tab + Smem::tab_pdot, *psum_s = tab + Smem::tab_psum;
        uint32_t inst_seq = 0;
        int cur_inst = -1, pre_inst = -1;
        const int sumM = P.sumM, Mmax = P.Mmax;
        const int Cp = (C + 3) & ~3;                           // label stride of the tables in shared memory
        const bool pair_st = (Mmax & 1) == 0 && ((uintptr_t)prm.acc_out & 7) == 0;
        // this instance's tables travel through registers so that the loads of the next instance are in flight
        // while the current one is processed
        float pre_rec[1024 / kEpiThreads], pre_bias = 0.f, pre_pdot[256 / kEpiThreads], pre_psum = 0.f;
        auto fetch_tab = [&](int inst) {
#pragma unroll
            for (int q = 0; q < 1024 / kEpiThreads; ++q) {
                const int k = q * kEpiThreads + et;
                pre_rec[q] = k < sumM * C ? P.recall[(int64_t)inst * sumM * C + k] : 0.f;
            }
            pre_bias = et < A * C ? P.bias[(int64_t)inst * A * C + et] : 0.f;
            if (PRIOR) {
#pragma unroll
                for (int q = 0; q < 256 / kEpiThreads; ++q) {
                    const int k = q * kEpiThreads + et;
                    pre_pdot[q] = k < sumM ? P.prior_dot[(int64_t)inst * sumM + k] : 0.f;
                }
                pre_psum = et < A ? P.prior_sum[inst * A + et] : 0.f;
            }
            pre_inst = inst;
        };
        // Descriptors travel two of the group's tiles ahead and the application of this thread's row one tile ahead,
        // so that no load of the loop waits for the result of another one issued in the same iteration.
        const int t0 = t_begin + eg;
        int4 d = t0 < t_end ? prm.tiles[t0] : make_int4(-1, 0, 0, 0);
        int4 d_n = t0 + kEpiGroups < t_end ? prm.tiles[t0 + kEpiGroups] : make_int4(-1, 0, 0, 0);
        int a_cur = (d.x >= 0 && row < d.z) ? tb.app[(int64_t)d.w + row] : 0;
        for (int t = t0; t < t_end; t += kEpiGroups) {
            if (d.x < 0) break;                                // valid tiles form a prefix of the block's range
            const int inst = d.x, rows = d.z;
            const int64_t req = (int64_t)d.w + row;
            const int a = min(max(a_cur, 0), A - 1);
            a_cur = (d_n.x >= 0 && row < d_n.z) ? tb.app[(int64_t)d_n.w + row] : 0;
            d = d_n;
            d_n = t + 2 * kEpiGroups < t_end ? prm.tiles[t + 2 * kEpiGroups] : make_int4(-1, 0, 0, 0);
            if (inst != cur_inst) {
                if (pre_inst != inst) fetch_tab(inst);
                mbar_arrive(bar(bar_epi_a(eg)));
                if (!warp_wait(bar(bar_epi_a(eg)), inst_seq & 1, abort_flag)) break;
#pragma unroll
                for (int q = 0; q < 1024 / kEpiThreads; ++q) {
                    const int k = q * kEpiThreads + et;
                    if (k < sumM * C) { const int g = k / C; tab[Smem::tab_recall + g * Cp + (k - g * C)] = pre_rec[q]; }
                }
                if (et < A * C) { const int g = et / C; tab[Smem::tab_bias + g * Cp + (et - g * C)] = pre_bias * kLog2e; }
                if (PRIOR) {
#pragma unroll
                    for (int q = 0; q < 256 / kEpiThreads; ++q) {
                        const int k = q * kEpiThreads + et;
                        if (k < sumM) tab[Smem::tab_pdot + k] = pre_pdot[q];
                    }
                    if (et < A) tab[Smem::tab_psum + et] = pre_psum;
                }
                mbar_arrive(bar(bar_epi_b(eg)));
                if (!warp_wait(bar(bar_epi_b(eg)), inst_seq & 1, abort_flag)) break;
                ++inst_seq;
                cur_inst = inst;
                if (inst + 1 < P.I) fetch_tab(inst + 1);
            }
            const bool valid = row < rows;
            const uint32_t acc_use = (uint32_t)(t - t_begin) >> 1;      // earlier uses of accumulator eg
            if (!warp_wait(bar(bar_acc_full(eg)), acc_use & 1, abort_flag)) break;
            tc_fence_after();
            const uint32_t taddr = tmem + ((uint32_t)(quad * 32) << 16) + (uint32_t)(eg * kAccCols);
            float z[CT];
#pragma unroll
            for (int c = 0; c < CT; ++c) z[c] = 0.f;
            for (int ap = 0; ap < A; ++ap) {
                if (__ballot_sync(0xffffffffu, a == ap) == 0) continue;
                float r1[CT];
                tmem_ld<CT>(taddr + (uint32_t)(ap * C), r1);
                tmem_wait_ld();
                if (a == ap) {
#pragma unroll
                    for (int c = 0; c < CT; ++c) z[c] = r1[c];
                }
            }
            tc_fence_before();
            mbar_arrive(bar(bar_acc_empty(eg)));

            // ---- softmax over the C labels of this row's application (base 2: log2(e) is in W and the bias)
            const float *bs = bias_s + a * Cp;
#pragma unroll
            for (int c = 0; c < CT; c += 4)
                if (c < C) {
                    const float4 bv = *reinterpret_cast<const float4 *>(bs + c);
                    z[c] += bv.x; z[c + 1] += bv.y; z[c + 2] += bv.z; z[c + 3] += bv.w;
                }
            float m = -INFINITY;
#pragma unroll
            for (int c = 0; c < CT; ++c)
                if (c < C) m = fmaxf(m, z[c]);
            float ssum = 0.f;
#pragma unroll
            for (int c = 0; c < CT; ++c) { z[c] = c < C ? exp2_unit(z[c] - m) : 0.f; ssum += z[c]; }
            const float inv = 1.f / ssum;
            // ---- Eq. 9 with the Dirichlet posterior mean; Eq. 12's variance from sums of differences to acc_0
            const int g0 = P.mfirst[a], M = P.mfirst[a + 1] - g0;
            float *dst = tb.acc32 + req * Mmax;
            float *dst2 = prm.acc_out ? prm.acc_out + req * Mmax : nullptr;
            float a0 = 0.f, s1 = 0.f, s2 = 0.f;
            // two models per pass: their recall rows are loaded together and accumulate in four independent chains
#pragma unroll 1
            for (int j = 0; j < Mmax; j += 2) {
                float aj0 = 0.f, aj1 = 0.f;
                const bool m0 = j < M, m1 = j + 1 < M;
                if (m0) {
                    const float *ra = recall_s + (g0 + j) * Cp, *rb = m1 ? ra + Cp : ra;
                    float p0 = 0.f, p1 = 0.f, q0 = 0.f, q1 = 0.f;
#pragma unroll
                    for (int c = 0; c < CT; c += 4)
                        if (c < C) {
                            const float4 rv = *reinterpret_cast<const float4 *>(ra + c);
                            const float4 sv = *reinterpret_cast<const float4 *>(rb + c);
                            p0 = fmaf(z[c], rv.x, p0); p1 = fmaf(z[c + 1], rv.y, p1);
                            q0 = fmaf(z[c], sv.x, q0); q1 = fmaf(z[c + 1], sv.y, q1);
                            p0 = fmaf(z[c + 2], rv.z, p0); p1 = fmaf(z[c + 3], rv.w, p1);
                            q0 = fmaf(z[c + 2], sv.z, q0); q1 = fmaf(z[c + 3], sv.w, q1);
                        }
                    aj0 = (p0 + p1) * inv;
                    aj1 = (q0 + q1) * inv;
                    if (PRIOR) {
                        aj0 = (pdot_s[g0 + j] + P.kappa * aj0) / (psum_s[a] + P.kappa);
                        if (m1) aj1 = (pdot_s[g0 + j + 1] + P.kappa * aj1) / (psum_s[a] + P.kappa);
                    }
                    if (j == 0) a0 = aj0;
                    const float d0 = aj0 - a0;
                    s1 += d0; s2 = fmaf(d0, d0, s2);
                    if (m1) {
                        const float d1 = aj1 - a0;
                        s1 += d1; s2 = fmaf(d1, d1, s2);
                    } else aj1 = 0.f;
                }
                if (valid) {
                    if (pair_st) {                             // rows of an even number of floats: 8-byte stores
                        *reinterpret_cast<float2 *>(dst + j) = make_float2(aj0, aj1);
                        if (dst2) *reinterpret_cast<float2 *>(dst2 + j) = make_float2(aj0, aj1);
                    } else {
                        dst[j] = aj0;
                        if (j + 1 < Mmax) dst[j + 1] = aj1;
                        if (dst2) { dst2[j] = aj0; if (j + 1 < Mmax) dst2[j + 1] = aj1; }
                    }
                }
            }
            if (valid) {
                const float invM = 1.f / (float)M, md = s1 * invM;
                tb.v32[req] = 1.f + fmaxf(fmaf(s2, invM, -md * md), 0.f);
            }
        }
    }

    // ---- teardown
    tc_fence_before();
    __syncthreads();
    if (tid == 0 && *abort_flag) dev_error(&prm.flags[0], kDevLimit);
    if (warp == kMmaWarp) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

}  // namespace mma
}  // namespace sp
