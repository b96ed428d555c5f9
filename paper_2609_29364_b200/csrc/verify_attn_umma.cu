// Verification attention on the 5th-generation tensor cores (tcgen05 + TMEM + TMA), for the
// shapes with many stacked query rows (large gamma), where the mma.sync kernel is bound by its
// own instruction stream rather than by HBM.
//
// Same operation and same split-KV bookkeeping as verify_attn.cu (Appendix G.2: anchor +
// proposal rows of a request attend its paged KV; Section 3: block maps), different engine.
//
// "Rows on lanes".  For one (request chunk, kv head) the M = G * (gamma + 1) <= 64 stacked query
// rows sit on TMEM lanes 0..M-1 and a tile of 128 keys on the columns:
//     S[rows x 128 keys]  = Q[rows x 128 dims] K^T     A = Q (shared, K-major, 128-byte swizzle), B = K tile (K-major)
//     O[rows x 128 dims] += P[rows x 128 keys] V       A = P (TMEM, bf16 pairs in S's own columns), B = V tile (MN-major)
// Both are UMMA M = 128, N = 128: lanes M..127 compute on whatever the rows past the staged Q
// hold and are never read.  A softmax thread owns one row: its maximum and its sum need no
// cross-thread step, and P goes straight back into tensor memory as the next contraction's A
// operand -- no trip through shared memory, no proxy fence.
//
// One persistent CTA per SM, twelve warps, every role walks the same static list of work units
// (chunk item, kv head):
//   warps 0-1, 4-5  softmax: a thread owns one row and one half of the tile's 128 keys (warps 0, 1 the
//               first 64, warps 4, 5 the rest; warp w reaches TMEM lanes 32 (w & 3) .. +31).  Read the
//               scores, mask, half-tile maximum, exchange it with the row's other warp, running maximum
//               (refreshed only when a score outgrows it by 2^8: then the row of O is rescaled in TMEM,
//               rare), P = 2^(s - m) as bf16 over the first 64 columns of the same S buffer.  From a
//               unit's second tile on P is formed with the maximum as it stands while the exchange is
//               under way, and formed again in the rare case that the exchange moves the maximum.
//   warps 2-3 / 10-11  K producers / V producers, each pair into its own ring of 32 KiB stages, each warp bringing
//               half of every tile (one warp's copies top out near 40 GB/s).  A K tile is sixteen
//               TMA boxes of 16 keys x 64 dims (the 128-byte swizzle caps a box row at 64 dims, and the
//               contraction over dims wants all 128 keys of a 64-dim half at one pitch).  A V tile is
//               eight boxes of 16 keys x 128 dims, one per pool block, through a 3-D view of the slab
//               whose outer coordinate is the 64-dim half: P V contracts over keys, 16 = one block per
//               instruction, so a block's two halves may sit side by side.  Blocks past the chunk are
//               loaded out of bounds (zero fill).  The first K producer, which reaches a unit before
//               anybody else, also stages the unit's Q into one of two swizzled buffers.
//   warps 8-9   epilogue: read the unit's row of O out of TMEM (the next unit's P V may start as soon
//               as that is done), then O / sum into the output, or the unnormalised row with its
//               maximum and sum into the split-KV partial, beside the next unit's main loop.  (Warps
//               8, 9 reach the same TMEM lanes as warps 0, 1.)  Partials are merged by a small kernel
//               launched behind this one: a persistent CTA that merged as the last arriver held up
//               its own pipeline for longer than a whole unit takes.
//   warp 6      issues S = Q K^T into one of three TMEM score buffers as soon as K has landed and the
//               P V that read the buffer's previous P is complete.
//   warp 7      issues O += P V once P is published and V has landed; zeroes the V rows of slots that
//               hold no token first (0 x NaN must not reach O).  Two issuing threads because a
//               tcgen05.mma costs its thread ~85 cycles whatever its shape.
// Every mbarrier wait is bounded; on expiry the CTA raises an abort flag, all roles leave their
// loops, the producers wait (bounded) for the copies they still have in flight, STATUS_TIMEOUT is
// recorded, TMEM is freed and the kernel returns.
#include <cuda.h>
#include <cuda_bf16.h>

#include "nsd_internal.h"

namespace nsd {
namespace {

constexpr int kTileKeys = 128;
constexpr int kBlockSizeU = 16;                          // keys per pool block
constexpr int kBlocksPerTile = 8;
constexpr int kHalfBytes = kTileKeys * 128;              // [128 keys][64 dims] bf16 = 16 KiB
constexpr int kStageBytes = 2 * kHalfBytes;              // one K or one V tile: dims 0-63, dims 64-127
constexpr int kRowsMax = 64;                             // stacked query rows a unit may have
constexpr int kQHalfBytes = kRowsMax * 128;              // [64 rows][64 dims]
constexpr int kQBytes = 2 * kQHalfBytes;
constexpr int kKStages = 3, kVStages = 3;
constexpr int kSBufs = 3;                                // S buffers in tensor memory
// warps 0, 1 and 4, 5: softmax (keys 0-63 / 64-127 of a tile); 2, 3: K producers; 6, 7: issuers; 8, 9: epilogue; 10, 11: V producers
constexpr int kWarpK = 2, kWarpSmB = 4, kWarpS = 6, kWarpPV = 7, kWarpEpi0 = 8, kWarpV = 10;
constexpr int kThreads = 12 * 32;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kMaxSlack = 8.0f;                        // the running maximum may lag the true one by this much (log2 units)
constexpr uint32_t kSpinLimit = 1u << 20;                // wait slices of ~2 us each

// Shared memory: two Q buffers, the K ring, the V ring, then barriers and a few words.  The A descriptor of
// S = Q K^T spans 128 rows; rows 64..127 of a Q buffer alias whatever follows it (the other Q buffer, the K ring):
// those lanes are never read.
constexpr int kOffQ = 0;
constexpr int kOffK = kOffQ + 2 * kQBytes;
constexpr int kOffV = kOffK + kKStages * kStageBytes;
constexpr int kOffMl = kOffV + kVStages * kStageBytes;   // [2][64] float2: a unit's running maxima and sums, softmax -> epilogue
constexpr int kOffX = kOffMl + 2 * kRowsMax * 8;         // [2 tile parities][2 key halves][64] floats: half-tile maxima, softmax <-> softmax
constexpr int kOffBars = kOffX + 2 * 2 * kRowsMax * 4;
constexpr int kNumBars = 2 * kKStages + 2 * kVStages + 4 + 3 * kSBufs + 2 + 1 + 2 + 2;
constexpr int kOffMisc = kOffBars + kNumBars * 8;        // tmem base, abort flag
constexpr int kSmemBytes = kOffMisc + 16;
static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");
// Tensor memory: three S buffers (P aliases the first 64 columns of its S), so that the S issuer, the softmax and the
// P V issuer each work on a tile of their own, and one O accumulator.
constexpr int kTmemCols = 512, kTmemS = 0, kTmemO = kSBufs * 128, kTmemStride = 128;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// ---- mbarrier / fences -------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity), "r"(2000u)
        : "memory");
    return done != 0;
}
// Bounded wait.  try_wait parks the thread in hardware until the phase completes or a time slice (hinted at
// ~2 us) runs out, so waiting threads do not flood shared memory with polls; the slices are counted, and the
// wait gives up when the CTA's abort flag is raised or the budget is spent (then it raises the flag itself).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, uint32_t limit) {
    for (uint32_t i = 0; i < limit; ++i) {
        if (mbar_try(bar, parity)) return true;
        if (*abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// Named barrier of the two epilogue warps (id 1, 64 threads), with an OR-reduction so that they leave together.
__device__ __forceinline__ bool epi_bar_or(bool pred) {
    uint32_t out;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %1, 0;\n\tbarrier.red.or.pred p, 1, 64, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(out)
        : "r"((uint32_t)pred)
        : "memory");
    return out != 0;
}

// ---- TMA -----------------------------------------------------------------------------------------
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int32_t x, int32_t y, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int32_t x, int32_t y, int32_t z, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
                 ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar)
                 : "memory");
}

// ---- tcgen05 ---------------------------------------------------------------------------------------
// Shared-memory matrix descriptor: start address, leading / stride byte offsets (16-byte units),
// descriptor version 1, layout type (2 = 128-byte swizzle).
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t layout) {
    return (uint64_t)((saddr >> 4) & 0x3FFF) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16) |
           ((uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32) | ((uint64_t)1 << 46) | ((uint64_t)(layout & 7) << 61);
}
// Instruction descriptor, kind::f16: fp32 accumulate, bf16 A and B, majorness bits, N >> 3, M >> 4.
__device__ __forceinline__ uint32_t instr_desc(int M, int N, int a_mn_major, int b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn_major << 15) | ((uint32_t)b_mn_major << 16) |
           ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
// D[tmem] (+)= A[smem] B[smem]
__device__ __forceinline__ void umma_ss(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate)
        : "memory");
}
// D[tmem] (+)= A[tmem] B[smem]; A is K-major: lane = row, a 32-bit column holds two consecutive bf16 of K
__device__ __forceinline__ void umma_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t db, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(tmem_d), "r"(tmem_a), "l"(db), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 32 consecutive columns of this thread's TMEM lane (no wait: several loads may be in flight).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* r) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
}
// 16 columns, for the rare paths that must not cost the common one its registers
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* r) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* r) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t* r) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
        "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
        "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Tiles of the work unit u (chunk item u / Hkv, kv head u % Hkv).
struct Unit {
    AttnItem item;
    int head, n_blk, n_tiles;
};
__device__ __forceinline__ Unit load_unit(const AttnLaunch& a, int64_t u) {
    Unit w;
    w.item = a.items[u / a.shape.Hkv];
    w.head = (int)(u % a.shape.Hkv);
    w.n_blk = w.item.blk_end - w.item.blk_begin;
    w.n_tiles = (w.n_blk + kBlocksPerTile - 1) / kBlocksPerTile;
    return w;
}

__global__ void __launch_bounds__(kThreads, 1)
verify_attn_umma_kernel(const __grid_constant__ AttnLaunch a) {
    // All shared memory is dynamic (no static variables), so that the swizzled tiles start at the aligned base of the
    // CTA's window; the kernel refuses to run (status bit, no access) should the base ever not be 1024-byte aligned.
    extern __shared__ __align__(1024) unsigned char smem[];
    uint64_t* const bars = reinterpret_cast<uint64_t*>(smem + kOffBars);
    uint64_t* const k_full = bars;
    uint64_t* const k_empty = k_full + kKStages;
    uint64_t* const v_full = k_empty + kKStages;
    uint64_t* const v_empty = v_full + kVStages;
    uint64_t* const q_full = v_empty + kVStages;      // [2]
    uint64_t* const q_empty = q_full + 2;             // [2]
    uint64_t* const s_full = q_empty + 2;             // [3]  S of a tile is complete
    uint64_t* const p_full = s_full + kSBufs;         // [3]  both softmax warps have written P over it
    uint64_t* const p_empty = p_full + kSBufs;        // [3]  the P V that read this buffer's P is complete
    uint64_t* const sm_done = p_empty + kSBufs;       // [2]  by unit parity: the softmax warps have left the unit's row statistics
    uint64_t* const o_full = sm_done + 2;             // [1]  one phase per unit: its last P V is complete
    uint64_t* const o_empty = o_full + 1;             // [2]  by unit parity: the epilogue has read the accumulator and the statistics
    uint64_t* const pair_bar = o_empty + 2;           // [2]  per row quadrant: the two softmax warps that share its rows meet
    uint32_t& tmem_base_s = *reinterpret_cast<uint32_t*>(smem + kOffMisc);
    volatile int& abort_s = *reinterpret_cast<volatile int*>(smem + kOffMisc + 4);
    float2* const ml_s = reinterpret_cast<float2*>(smem + kOffMl);
    float* const xmax_s = reinterpret_cast<float*>(smem + kOffX);
    if ((smem_u32(smem) & 1023u) != 0) {
        if (threadIdx.x == 0) atomicOr(a.status, STATUS_LAYOUT);
        return;
    }

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // every unit has its own draft depth: item.gamma + 1 query rows per head, M = G * (item.gamma + 1) stacked rows
    const int Hkv = a.shape.Hkv, Hq = a.shape.Hq, G = Hq / Hkv, MS = a.m_stride;
    const int64_t n_units = (int64_t)a.n_items * Hkv;
    const uint32_t smem0 = smem_u32(smem);
    const uint32_t wait_limit = a.wait_budget ? a.wait_budget : kSpinLimit;

    if (tid == 0) {
        // two producer warps arm each stage, each with its half of the bytes
        for (int s = 0; s < kKStages; ++s) mbar_init(smem_u32(&k_full[s]), 2), mbar_init(smem_u32(&k_empty[s]), 1);
        for (int s = 0; s < kVStages; ++s) mbar_init(smem_u32(&v_full[s]), 2), mbar_init(smem_u32(&v_empty[s]), 1);
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&q_full[b]), 1);
            mbar_init(smem_u32(&q_empty[b]), 1);
        }
        for (int b = 0; b < kSBufs; ++b) {
            mbar_init(smem_u32(&s_full[b]), 1);
            mbar_init(smem_u32(&p_full[b]), 4);
            mbar_init(smem_u32(&p_empty[b]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&sm_done[b]), 4);
            mbar_init(smem_u32(&o_empty[b]), 2);
            mbar_init(smem_u32(&pair_bar[b]), 2);
        }
        mbar_init(smem_u32(o_full), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        abort_s = 0;
    }
    // the row sums of the statistics are accumulated with atomic adds and start at zero
    if (tid < 2 * kRowsMax) ml_s[tid] = make_float2(0.f, 0.f);
    // rows past M of both Q buffers stay zero for the whole kernel (the stager writes rows < M only)
    for (int c = tid; c < 2 * kQBytes / 16; c += kThreads) reinterpret_cast<int4*>(smem + kOffQ)[c] = make_int4(0, 0, 0, 0);
    fence_async_smem();
    if (warp == kWarpS) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "n"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_s = tmem_base_s + kTmemS, tmem_o = tmem_base_s + kTmemO;
    if (warp == kWarpK || warp == kWarpK + 1 || warp == kWarpV || warp == kWarpV + 1) {
        // ================================ producers ================================
        // Two warps per ring, each bringing half of every tile: one warp's copies move at most ~40 GB/s, whatever
        // their number in flight, and an SM's share of HBM is more than that per ring.
        const bool is_v = warp >= kWarpV;
        const int part = (warp - (is_v ? kWarpV : kWarpK));                    // which half of the tile this warp brings
        const int n_stages = is_v ? kVStages : kKStages;
        uint64_t* full = is_v ? v_full : k_full;
        uint64_t* empty = is_v ? v_empty : k_empty;
        const uint32_t ring = smem0 + (is_v ? kOffV : kOffK);
        const int32_t rows_per_kv = Hkv * kBlockSizeU;                        // rows between the K and the V tile of a block
        const int32_t oob_row = a.shape.num_blocks * 2 * rows_per_kv;         // past the slab: zero fill
        // K: warp = 64-dim half, lane = block of the tile: 8 boxes of 2 KiB.  V: warp = blocks 0-3 / 4-7 of the tile; with the
        // 3-D map lane = block, 4 boxes of 4 KiB, else lane = (block, half), 8 boxes of 2 KiB.
        const bool big = is_v && a.tmap3_valid;
        const int n_lanes = big ? 4 : 8;
        const int b = is_v ? (big ? part * 4 + lane : part * 4 + (lane >> 1)) : lane;
        const int half = is_v ? (big ? 0 : lane & 1) : part;
        const bool stages_q = !is_v && part == 0;
        uint32_t g = 0;
        bool ok = true;
        uint32_t uidx = 0;
        // The first K producer, which runs up to three tiles ahead of the S issuer and so reaches a unit first, also
        // stages the units' Q -- [64 rows][64 dims] per half, 128-byte swizzle; row m = i * G + h is query row i of head
        // head * G + h; rows past M were zeroed once.  The rows go global -> shared by cp.async (no registers held),
        // started a few tiles into the unit BEFORE the one they belong to, when the buffer's previous user is surely
        // done, and collected at the unit boundary.
        auto q_start = [&](const Unit& w, uint32_t k) -> bool {                 // Q of this CTA's unit number k
            const int qb = k & 1;
            // the last S of the unit that used this buffer is complete
            bool okq = true;
            if (lane == 0 && k >= 2 && !mbar_wait(smem_u32(&q_empty[qb]), ((k >> 1) - 1) & 1, &abort_s, wait_limit)) okq = false;
            okq = __shfl_sync(0xffffffffu, (int)okq, 0) != 0;
            if (!okq) return false;
            // rows past this unit's M keep whatever an earlier unit left there: finite values on lanes nobody reads
            const int64_t row_base = w.item.row0;
            const int M = G * (w.item.gamma + 1);
            const uint32_t qdst = smem0 + kOffQ + qb * kQBytes;
            for (int c = lane; c < M * 16; c += 32) {
                const int m = c >> 4, ch = c & 15, hh = ch >> 3, cc = ch & 7;
                const int i = m / G, h = m - i * G;
                const uint16_t* src = a.q + ((row_base + i) * Hq + w.head * G + h) * 128 + ch * 8;
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(qdst + hh * kQHalfBytes + m * 128 + ((cc ^ (m & 7)) << 4)), "l"(src) : "memory");
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
            return true;
        };
        auto q_finish = [&](uint32_t k) {
            asm volatile("cp.async.wait_group 0;" ::: "memory");
            fence_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&q_full[k & 1]));
        };
        if (stages_q && (int64_t)blockIdx.x < n_units) ok = q_start(load_unit(a, blockIdx.x), 0);
        for (int64_t u = blockIdx.x; u < n_units && ok; u += gridDim.x, ++uidx) {
            const Unit w = load_unit(a, u);
            const int r = w.item.req;
            if (stages_q) q_finish(uidx);
            const bool q_next = stages_q && u + gridDim.x < n_units;
            const int q_tile = min(3, w.n_tiles - 1);                          // the tile after which the next unit's Q is started
            const int32_t* table = a.kv_indices + (int64_t)w.item.tbl_off + w.item.blk_begin;   // the plan copied kv_indptr[r] into the item
            // block ids are read one tile ahead, so the table's latency hides behind the current tile's wait and issue
            int32_t blk_next = (lane < n_lanes && b < w.n_blk) ? __ldg(table + b) : -1;
            for (int t = 0; t < w.n_tiles; ++t, ++g) {
                const uint32_t stage = g % n_stages, use = g / n_stages;
                const int bi = t * kBlocksPerTile + b;
                int32_t row = oob_row;
                int32_t blk = blk_next;
                blk_next = (lane < n_lanes && bi + kBlocksPerTile < w.n_blk) ? __ldg(table + bi + kBlocksPerTile) : -1;
                if (lane < n_lanes && bi < w.n_blk) {
                    if ((uint32_t)blk >= (uint32_t)a.shape.num_blocks) {
                        atomicOr(a.status, STATUS_BAD_BLOCK);
                        atomicCAS(a.status + 1, 0, r + 1);
                        blk = 0;
                    }
                    row = blk * 2 * rows_per_kv + w.head * kBlockSizeU + (is_v ? rows_per_kv : 0);
                }
                if (lane == 0) {
                    if (use > 0 && !mbar_wait(smem_u32(&empty[stage]), (use - 1) & 1, &abort_s, wait_limit)) ok = false;
                    if (ok) mbar_expect_tx(smem_u32(&full[stage]), kStageBytes / 2);
                }
                ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
                if (!ok) break;
                if (q_next && t == q_tile) ok = q_start(load_unit(a, u + gridDim.x), uidx + 1);
                if (!ok) break;
                if (big) {
                    if (lane < 4) tma_load_3d(ring + stage * kStageBytes + b * 4096, &a.tmap3, 0, row, 0, smem_u32(&full[stage]));
                } else if (lane < 8) {
                    const uint32_t dst = is_v ? b * 4096 + half * 2048 : half * kHalfBytes + b * 2048;   // V: a block's halves side by side
                    tma_load_2d(ring + stage * kStageBytes + dst, &a.tmap, half * 64, row, smem_u32(&full[stage]));
                }
            }
        }
        __syncwarp();
        if (abort_s && lane == 0) {
            // the CTA is giving up: the tiles this warp armed and nobody consumed may still be landing; give each stage's
            // latest phase a bounded wait of its own before the shared memory goes back to the SM
            for (uint32_t back = 0; back < (uint32_t)n_stages && back < g; ++back) {
                const uint32_t gg = g - 1 - back;
                for (uint32_t i = 0; i < wait_limit; ++i)
                    if (mbar_try(smem_u32(&full[gg % n_stages]), (gg / n_stages) & 1)) break;
            }
        }
    } else if (warp == kWarpS) {
        // ================================ S issuer ================================
        if (lane == 0) {
            const uint32_t idesc_qk = instr_desc(128, 128, 0, 0);
            uint32_t g = 0, uidx = 0;
            bool ok = true;
            for (int64_t u = blockIdx.x; u < n_units && ok; u += gridDim.x, ++uidx) {
                const Unit w = load_unit(a, u);
                const int qb = uidx & 1;
                if (!mbar_wait(smem_u32(&q_full[qb]), (uidx >> 1) & 1, &abort_s, wait_limit)) break;
                const uint32_t q_s = smem0 + kOffQ + qb * kQBytes;
                for (int t = 0; t < w.n_tiles; ++t, ++g) {
                    const uint32_t ks = g % kKStages, sb = g % kSBufs;
                    // K has landed; the P V that read P out of this score buffer three tiles ago is complete
                    if (!mbar_wait(smem_u32(&k_full[ks]), (g / kKStages) & 1, &abort_s, wait_limit) ||
                        (g >= kSBufs && !mbar_wait(smem_u32(&p_empty[sb]), ((g / kSBufs) - 1) & 1, &abort_s, wait_limit))) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t kb = smem0 + kOffK + ks * kStageBytes;
#pragma unroll
                    for (int k = 0; k < 8; ++k) {               // 8 steps of 16 dims, 64 dims per swizzled half
                        const uint64_t da = smem_desc(q_s + (k >> 2) * kQHalfBytes + (k & 3) * 32, 16, 1024, 2);
                        const uint64_t db = smem_desc(kb + (k >> 2) * kHalfBytes + (k & 3) * 32, 16, 1024, 2);
                        umma_ss(tmem_s + sb * kTmemStride, da, db, idesc_qk, k > 0);
                    }
                    umma_commit(smem_u32(&k_empty[ks]));
                    umma_commit(smem_u32(&s_full[sb]));
                    if (t == w.n_tiles - 1) umma_commit(smem_u32(&q_empty[qb]));
                }
            }
        }
        __syncwarp();
    } else if (warp == kWarpPV) {
        // ================================ P V issuer ================================
        const uint32_t idesc_pv = instr_desc(128, 128, 0, 1);
        uint32_t g = 0, uidx = 0;
        bool ok = true;
        for (int64_t u = blockIdx.x; u < n_units && ok; u += gridDim.x, ++uidx) {
            const Unit w = load_unit(a, u);
            const int n_total = w.item.ctx + w.item.gamma + 1;
            // the epilogue has read the previous unit out of the accumulator
            if (lane == 0 && uidx >= 1 && !mbar_wait(smem_u32(&o_empty[(uidx - 1) & 1]), ((uidx - 1) >> 1) & 1, &abort_s, wait_limit)) ok = false;
            ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
            for (int t = 0; t < w.n_tiles && ok; ++t, ++g) {
                const uint32_t vs = g % kVStages, sb = g % kSBufs;
                if (lane == 0 && !mbar_wait(smem_u32(&v_full[vs]), (g / kVStages) & 1, &abort_s, wait_limit)) ok = false;
                ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
                if (!ok) break;
                // slots that hold no token may carry anything in the pool: their V row must be finite for 0 * V
                const int key0 = w.item.blk_begin * kBlockSizeU + t * kTileKeys;
                const int z0 = max(n_total - key0, 0), z1 = min(w.item.blk_end * kBlockSizeU - key0, kTileKeys);
                if (z0 < z1) {
                    unsigned char* vt = smem + kOffV + vs * kStageBytes;
                    for (int c = lane; c < (z1 - z0) * 16; c += 32) {
                        const int row = z0 + (c >> 4), ch = c & 15;               // key `row` of the tile: block row >> 4, slot row & 15
                        *reinterpret_cast<int4*>(vt + (row >> 4) * 4096 + (ch >> 3) * 2048 + (row & 15) * 128 + (ch & 7) * 16) = make_int4(0, 0, 0, 0);
                    }
                    fence_async_smem();
                    __syncwarp();
                }
                if (lane == 0) {
                    if (!mbar_wait(smem_u32(&p_full[sb]), (g / kSBufs) & 1, &abort_s, wait_limit)) {
                        ok = false;
                    } else {
                        tc_fence_after();
                        const uint32_t vb = smem0 + kOffV + vs * kStageBytes;
                        const uint32_t p_t0 = tmem_s + sb * kTmemStride;
#pragma unroll
                        for (int k = 0; k < 8; ++k) {           // 8 steps of 16 keys = one pool block = 8 columns of bf16 pairs
                            // a block's V: [half][16 keys][64 dims]; halves 2 KiB apart (LBO), 8-key groups 1 KiB apart (SBO)
                            const uint64_t db = smem_desc(vb + k * 4096, 2048, 1024, 2);
                            umma_ts(tmem_o, p_t0 + k * 8, db, idesc_pv, (t > 0 || k > 0) ? 1u : 0u);
                        }
                        umma_commit(smem_u32(&v_empty[vs]));
                        umma_commit(smem_u32(&p_empty[sb]));
                        if (t == w.n_tiles - 1) umma_commit(smem_u32(o_full));
                    }
                }
                ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
            }
        }
        __syncwarp();
    } else if (warp < 2 || warp == kWarpSmB || warp == kWarpSmB + 1) {
        // ================================ softmax ================================
        // Thread = one stacked query row (TMEM lane 32 q + lane, q = warp & 3) and one half of the tile's keys: warps 0, 1
        // take keys 0-63, warps 4, 5 keys 64-127.  Row m = i * G + h sees keys [0, ctx + i].  Scores go to the log2 domain
        // with the 1/sqrt(d) scale folded into one FFMA.  The two warps of a row exchange their half-tile maxima through
        // shared memory (a bounded mbarrier rendezvous), so both hold the same running maximum and take the same
        // decisions; it is refreshed, and the row of O rescaled, only when a score exceeds it by more than 2^8.
        const int q = warp & 3;
        const bool is_b = warp >= kWarpSmB;
        const uint32_t lane_base = (uint32_t)(q * 32) << 16;
        const uint32_t col0 = is_b ? 64u : 0u;              // this warp's score columns, and dims of O in a rescale
        const float sc = rsqrtf(128.f) * kLog2e;
        const int m_row = q * 32 + lane;
        uint32_t g = 0, uidx = 0;
        uint32_t pair_n = 0;                                // meetings of the row's two warps so far (one per tile, rarely two)
        bool fail = false;                                  // warp-uniform: a wait gave up (the CTA is aborting)
        for (int64_t u = blockIdx.x; u < n_units && !fail; u += gridDim.x, ++uidx) {
            const Unit w = load_unit(a, u);
            const int mr = uidx & 1;                        // which entry of the row statistics this unit uses
            const int ctx = w.item.ctx;                     // the plan's copy: no dependent load at a unit boundary
            const int chunk_end = w.item.blk_end * kBlockSizeU;
            const int gamma = w.item.gamma;
            const bool live = m_row < G * (gamma + 1);      // lanes past the unit's rows hold no row and are never read
            // keys this row may see: [0, vis_stop)
            const int vis_stop = live ? min(ctx + min(m_row / G, gamma) + 1, chunk_end) : 0x3fffffff;   // lanes without a row never mask
            float m_run = -INFINITY, l_run = 0.f;           // l_run: this warp's half of the keys only
            for (int t = 0; t < w.n_tiles && !fail; ++t, ++g) {
                const uint32_t sb = g % kSBufs;
                const uint32_t tmem_sb = tmem_s + sb * kTmemStride + lane_base;
                if (!mbar_wait(smem_u32(&s_full[sb]), (g / kSBufs) & 1, &abort_s, wait_limit)) fail = true;
                fail = __any_sync(0xffffffffu, fail);
                if (fail) break;
                tc_fence_after();
                uint32_t sr[64];
                const int key0 = w.item.blk_begin * kBlockSizeU + t * kTileKeys + (int)col0;
                const int n_vis = vis_stop - key0;          // visible keys of this half tile for this row (may be <= 0 or >= 64)
                const bool masked = __any_sync(0xffffffffu, n_vis < 64);
                // this half's scores: tensor memory -> registers, hidden keys replaced
                auto load_scores = [&]() {
                    tmem_ld32(tmem_sb + col0, sr);
                    tmem_ld32(tmem_sb + col0 + 32, sr + 32);
                    tmem_wait_ld();
                    // Lanes past M hold no row: they take part in the tensor-memory loads and stores (which are warp-wide) but
                    // sit out the arithmetic, so a warp with few rows costs few lanes' worth of energy.
                    if (live && masked) {
                        // keys past the chunk (zero-filled boxes) belong to nobody, keys past ctx + i are hidden from row i,
                        // and slots past the last token may hold anything: all replaced by -inf with a select
#pragma unroll
                        for (int j = 0; j < 64; ++j) sr[j] = j < n_vis ? sr[j] : 0xff800000u;
                    }
                };
                // P = 2^(s * sc - m), bf16 pairs, over the scores in place: the 64 keys become 32 words
                float l0 = 0.f, l1 = 0.f;
                auto weights = [&]() {
                    const float nm = m_run == -INFINITY ? 0.f : -m_run;
                    l0 = 0.f, l1 = 0.f;
                    if (live) {
#pragma unroll
                        for (int j = 0; j < 64; j += 2) {
                            const float p0 = ex2_approx(fmaf(__uint_as_float(sr[j]), sc, nm));
                            const float p1 = ex2_approx(fmaf(__uint_as_float(sr[j + 1]), sc, nm));
                            l0 += p0;
                            l1 += p1;
                            sr[j >> 1] = pack_bf16(p0, p1);
                        }
                    }
                };
                load_scores();
                float mx0 = -INFINITY, mx1 = -INFINITY;
                if (live) {
#pragma unroll
                    for (int j = 0; j < 64; j += 2) {
                        mx0 = fmaxf(mx0, __uint_as_float(sr[j]));
                        mx1 = fmaxf(mx1, __uint_as_float(sr[j + 1]));
                    }
                }
                // ---- both halves' maxima: mine out, and an arrival that also tells the row's other warp that my scores are
                //      in registers.  The running maximum moves rarely (only when a score outgrows it by 2^8), so from a
                //      unit's second tile on the weights are formed with the maximum as it stands while the other half's
                //      arrival is on its way, and formed again in the rare case that the exchange does move the maximum.
                float* xm = xmax_s + (pair_n & 1) * (2 * kRowsMax);
                const float mine = fmaxf(mx0, mx1);
                xm[(is_b ? kRowsMax : 0) + m_row] = mine;
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&pair_bar[q]));
                const bool ahead = t > 0;
                if (ahead) weights();
                if (!mbar_wait(smem_u32(&pair_bar[q]), pair_n & 1, &abort_s, wait_limit)) fail = true;
                fail = __any_sync(0xffffffffu, fail);
                if (fail) break;
                ++pair_n;
                const float m_tile = fmaxf(mine, xm[(is_b ? 0 : kRowsMax) + m_row]) * sc;   // -inf when the row sees nothing of this tile
                const bool outgrown = live && m_tile > m_run + kMaxSlack;      // also the first visible key (m_run = -inf)
                const bool moved = __any_sync(0xffffffffu, outgrown);          // the same answer in both warps of the rows: same rows, same numbers
                if (moved) {
                    const float m_new = outgrown ? m_tile : m_run;
                    // m_run = -inf: nothing accumulated yet, the factor is irrelevant but must not be NaN
                    const float resc = (outgrown && m_run != -INFINITY) ? ex2_approx(m_run - m_new) : (outgrown ? 0.f : 1.f);
                    if (t > 0) {
                        // O holds this unit's earlier tiles, complete once P V of tile g - 1 is; each warp of the pair rescales
                        // its 64 dims of the row
                        if (!mbar_wait(smem_u32(&p_empty[(g - 1) % kSBufs]), ((g - 1) / kSBufs) & 1, &abort_s, wait_limit)) fail = true;
                        fail = __any_sync(0xffffffffu, fail);
                        if (fail) break;
                        tc_fence_after();
                        const uint32_t tmem_ob = tmem_o + lane_base + col0;
#pragma unroll 1
                        for (int c = 0; c < 4; ++c) {
                            uint32_t x[16];
                            tmem_ld16(tmem_ob + c * 16, x);
                            tmem_wait_ld();
#pragma unroll
                            for (int j = 0; j < 16; ++j) x[j] = __float_as_uint(__uint_as_float(x[j]) * resc);
                            tmem_st16(tmem_ob + c * 16, x);
                        }
                        tmem_wait_st();
                    }
                    l_run *= resc;
                    m_run = m_new;
                }
                if (moved || !ahead) {
                    if (ahead) {
                        // the weights formed ahead are void: the scores again (nobody has written P over them yet: a warp
                        // stores after this point only), and a second meeting so that the other warp's P, which lands on
                        // columns this warp's scores occupy, waits for this load
                        load_scores();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(smem_u32(&pair_bar[q]));
                        if (!mbar_wait(smem_u32(&pair_bar[q]), pair_n & 1, &abort_s, wait_limit)) fail = true;
                        fail = __any_sync(0xffffffffu, fail);
                        if (fail) break;
                        ++pair_n;
                    }
                    weights();
                }
                l_run += l0 + l1;
                tmem_st32(tmem_sb + (col0 >> 1), sr);
                tmem_wait_st();
                if (t == w.n_tiles - 1) {
                    // the epilogue of the unit before last has read (and cleared) this entry of the statistics
                    if (uidx >= 2 && !mbar_wait(smem_u32(&o_empty[mr]), ((uidx >> 1) - 1) & 1, &abort_s, wait_limit)) fail = true;
                    fail = __any_sync(0xffffffffu, fail);
                    if (fail) break;
                    if (!is_b) ml_s[mr * kRowsMax + m_row].x = m_run;
                    atomicAdd(&ml_s[mr * kRowsMax + m_row].y, l_run);          // two addends onto zero: the order cannot matter
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(smem_u32(&p_full[sb]));
                    if (t == w.n_tiles - 1) mbar_arrive(smem_u32(&sm_done[mr]));
                }
            }
        }
    } else {
        // ================================ epilogue (warps 8, 9) ================================
        // Thread = one row (TMEM lane te) of O.
        const int te = tid - kWarpEpi0 * 32;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        uint32_t uidx = 0;
        for (int64_t u = blockIdx.x; u < n_units; u += gridDim.x, ++uidx) {
            const Unit w = load_unit(a, u);
            const int mr = uidx & 1;
            const int head = w.head;
            const int64_t row_base = w.item.row0;
            const bool live = te < G * (w.item.gamma + 1);
            const bool mine = mbar_wait(smem_u32(o_full), uidx & 1, &abort_s, wait_limit) &&
                              mbar_wait(smem_u32(&sm_done[mr]), (uidx >> 1) & 1, &abort_s, wait_limit);
            if (epi_bar_or(!mine)) break;                   // a wait gave up: both warps leave together
            tc_fence_after();
            const float2 ml = ml_s[mr * kRowsMax + te];
            ml_s[mr * kRowsMax + te] = make_float2(0.f, 0.f);                  // ready for the unit after next
            const bool split = w.item.part_base >= 0;
            const int64_t slot = split ? ((int64_t)w.item.part_base + w.item.chunk_idx) * Hkv + head : 0;
            const int i = te / G, h = te - i * G;
            const int64_t orow = (row_base + i) * Hq + head * G + h;
            const float inv = 1.f / ml.y;
            // the row leaves tensor memory in two halves of 64 dims; the next unit's P V may start once the second is out
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                uint32_t x[64];
                tmem_ld32(tmem_o + lane_base + hh * 64, x);
                tmem_ld32(tmem_o + lane_base + hh * 64 + 32, x + 32);
                tmem_wait_ld();
                if (hh == 1) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&o_empty[mr]));
                }
                if (live) {
                    if (split) {
                        float4* pa = reinterpret_cast<float4*>(a.part_acc + (slot * MS + te) * 128 + hh * 64);
#pragma unroll
                        for (int j = 0; j < 16; ++j)
                            pa[j] = make_float4(__uint_as_float(x[4 * j]), __uint_as_float(x[4 * j + 1]), __uint_as_float(x[4 * j + 2]),
                                                __uint_as_float(x[4 * j + 3]));
                    } else {
                        uint4* po = reinterpret_cast<uint4*>(a.o + orow * 128 + hh * 64);
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            uint4 pk;
                            pk.x = pack_bf16(__uint_as_float(x[8 * j]) * inv, __uint_as_float(x[8 * j + 1]) * inv);
                            pk.y = pack_bf16(__uint_as_float(x[8 * j + 2]) * inv, __uint_as_float(x[8 * j + 3]) * inv);
                            pk.z = pack_bf16(__uint_as_float(x[8 * j + 4]) * inv, __uint_as_float(x[8 * j + 5]) * inv);
                            pk.w = pack_bf16(__uint_as_float(x[8 * j + 6]) * inv, __uint_as_float(x[8 * j + 7]) * inv);
                            po[j] = pk;
                        }
                    }
                }
            }
            if (live) {
                if (split) {
                    // a row that saw no key of this chunk (sum 0, maximum -inf) takes no part in the merge
                    *reinterpret_cast<float2*>(a.part_ml + (slot * MS + te) * 2) = ml;
                } else if (a.lse) {
                    a.lse[orow] = (ml.x + log2f(ml.y)) * 0.6931471805599453f;
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == kWarpS) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base_s), "n"(kTmemCols) : "memory");
    }
    if (tid == 0 && abort_s) atomicOr(a.status, STATUS_TIMEOUT);
}

// Merges the split-KV partials the kernel above left behind: one CTA per (work item, kv head), and only the CTA of a
// split request's first chunk has work -- it combines that (request, head)'s chunks in chunk order (deterministic) and
// writes the normalised rows.  Thread = one 4-dim column of one row at a time; blockIdx.y shares a (request, head)'s
// elements out over kMergeSlices CTAs, because a thread's elements are strictly one after another (two dependent passes
// over the chunks each) and the kernel is bound by that latency, not by its few megabytes.
constexpr int kMergeSlices = 3;
__global__ void __launch_bounds__(128)
verify_attn_umma_merge_kernel(const __grid_constant__ AttnLaunch a) {
    const int Hkv = a.shape.Hkv, Hq = a.shape.Hq, G = Hq / Hkv, MS = a.m_stride;
    const int item_idx = blockIdx.x / Hkv, head = blockIdx.x - item_idx * Hkv;
    const AttnItem it = a.items[item_idx];
    if (it.nchunks <= 1 || it.chunk_idx != 0) return;
    const int nch = it.nchunks;
    const int64_t slot0 = (int64_t)it.part_base * Hkv + head;                 // chunk c sits at slot0 + c * Hkv
    const int64_t row_base = it.row0;
    const int M = G * (it.gamma + 1);
    for (int e = blockIdx.y * 128 + threadIdx.x; e < M * 32; e += 128 * kMergeSlices) {
        const int m = e >> 5, d4 = e & 31;
        float mstar = -INFINITY;
        for (int c = 0; c < nch; ++c) mstar = fmaxf(mstar, __ldcg(a.part_ml + ((slot0 + (int64_t)c * Hkv) * MS + m) * 2));
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        float l = 0.f;
#pragma unroll 4
        for (int c = 0; c < nch; ++c) {
            const int64_t sl = slot0 + (int64_t)c * Hkv;
            const float2 mlc = __ldcg(reinterpret_cast<const float2*>(a.part_ml + (sl * MS + m) * 2));
            const float4 v = __ldcg(reinterpret_cast<const float4*>(a.part_acc + (sl * MS + m) * 128) + d4);
            // a row that saw no key of a chunk (sum 0, maximum -inf) takes no part
            const float wgt = mlc.x == -INFINITY ? 0.f : exp2f(mlc.x - mstar);
            acc.x += wgt * v.x;
            acc.y += wgt * v.y;
            acc.z += wgt * v.z;
            acc.w += wgt * v.w;
            l += wgt * mlc.y;
        }
        const float invl = 1.f / l;
        const int i = m / G, h = m - i * G;
        const int64_t orow = (row_base + i) * Hq + head * G + h;
        uint2 pk;
        pk.x = pack_bf16(acc.x * invl, acc.y * invl);
        pk.y = pack_bf16(acc.z * invl, acc.w * invl);
        *reinterpret_cast<uint2*>(a.o + orow * 128 + d4 * 4) = pk;
        if (a.lse && d4 == 0) a.lse[orow] = (mstar + log2f(l)) * 0.6931471805599453f;
    }
}

}  // namespace

cudaError_t attn_umma_init() {
    return cudaFuncSetAttribute(verify_attn_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
}

bool attn_umma_supported(const AttnLaunch& a) {
    return a.shape.D == 128 && a.shape.bs == 16 && a.m_rows >= 1 && a.m_rows <= kRowsMax && !a.fuse && a.tmap_valid;
}

// Where this engine is the faster one: from five 8-row tiles on (gamma >= 8 at the Qwen3-8B group size) the mma.sync
// kernel is bound by its own tensor-pipe chains and shared-memory reads, not by HBM.
bool attn_umma_preferred(const AttnLaunch& a) { return a.m_rows > 32; }

cudaError_t launch_attn_umma(const AttnLaunch& a, cudaStream_t stream, int n_sms) {
    if (a.n_items <= 0) return cudaSuccess;
    const int64_t n_units = (int64_t)a.n_items * a.shape.Hkv;
    const int grid = (int)(n_units < n_sms ? n_units : n_sms);
    verify_attn_umma_kernel<<<grid, kThreads, kSmemBytes, stream>>>(a);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess || !a.any_split) return e;
    verify_attn_umma_merge_kernel<<<dim3((unsigned)n_units, kMergeSlices), 128, 0, stream>>>(a);
    return cudaGetLastError();
}

// Tensor map over one layer slab seen as a 2-D bf16 tensor [rows][128 dims], rows = (block, K|V, kv head, slot);
// box = 16 rows x 64 dims with the 128-byte swizzle the UMMA descriptors expect.  Returns false when the driver
// entry point is unavailable or refuses the shape (the caller then stays on the mma.sync kernel).
bool make_kv_tensor_map(CUtensorMap* map, const void* slab, const Shape& s) {
    typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                 const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                 CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static EncodeFn encode = [] {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess)
            fn = nullptr;
        return reinterpret_cast<EncodeFn>(fn);
    }();
    if (!encode || s.D != 128 || s.bs != 16) return false;
    const cuuint64_t dims[2] = {128, (cuuint64_t)s.num_blocks * 2 * s.Hkv * 16};
    const cuuint64_t strides[1] = {256};
    const cuuint32_t box[2] = {64, 16};
    const cuuint32_t estr[2] = {1, 1};
    return encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(slab), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The same slab as a 3-D tensor [half = 2][rows][64 dims] -- the 64-dim half is the OUTER coordinate, 128 bytes apart --
// so that one box of 64 dims x 16 rows x 2 halves brings the whole [16 keys][128 dims] tile of a block, its halves side
// by side in shared memory.  Returns false when the driver refuses the view (the V producer then uses 2-D boxes).
bool make_kv_tensor_map3(CUtensorMap* map, const void* slab, const Shape& s) {
    typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                 const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                 CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static EncodeFn encode = [] {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess)
            fn = nullptr;
        return reinterpret_cast<EncodeFn>(fn);
    }();
    if (!encode || s.D != 128 || s.bs != 16) return false;
    const cuuint64_t dims[3] = {64, (cuuint64_t)s.num_blocks * 2 * s.Hkv * 16, 2};
    const cuuint64_t strides[2] = {256, 128};
    const cuuint32_t box[3] = {64, 16, 2};
    const cuuint32_t estr[3] = {1, 1, 1};
    return encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(slab), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace nsd
