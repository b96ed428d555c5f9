// Verification attention on the 5th-generation tensor cores (tcgen05 + TMEM + TMA).
//
// Same operation and same split-KV bookkeeping as verify_attn.cu (Appendix G.2: anchor +
// proposal rows of a request attend its paged KV; Section 3: block maps), different engine.
//
// "Keys on lanes".  A tile is 128 keys.  Both contractions put the long dimension on the 128
// TMEM lanes and the few query rows on the columns:
//     S^T[128 keys x R rows]  = K[128 x 128] Q^T            A = K tile (K-major, 128B swizzle), B = Q (K-major)
//     O^T[128 dims x R rows] += V^T[128 x 128 keys] P^T     A = V tile (MN-major), B = P^T (MN-major)
// so each of the 128 softmax threads owns one key (one TMEM lane) of S^T and each epilogue thread
// one output dimension of O^T.  R = rows padded to 32 / 48 / 64.  tcgen05.mma costs its issuing
// thread ~80 cycles whatever N is, so the instruction count per tile (8 + 8) is what matters.
//
// One persistent CTA per SM, 13 warps, every role walks the same static list of work units
// (chunk item, kv head):
//   warp 8 / warp 9   K producer / V producer: 16 lanes each issue one TMA box (16 keys x 64 dims,
//                     128-byte swizzle) per tile into their own ring of 32 KiB stages.  Two issuing
//                     warps because one warp's TMA issue rate tops out near 39 GB/s per SM; K stages
//                     are released as soon as S^T is computed, so the K stream runs up to three tiles
//                     ahead of V and P^T is usually ready when a V tile lands: almost the whole ring
//                     is in flight.  Blocks past the chunk are loaded out of bounds (zero fill).
//   warp 12           stages Q of the next unit into one of two swizzled Q buffers.
//   warp 10           issues S^T = K Q^T into one of three TMEM score buffers, as soon as K lands.
//   warp 11           issues O^T += V^T P^T once P^T is published and V has landed; zeroes V rows of
//                     slots that hold no token first (0 x NaN must not reach O^T).
//   warps 0-3         softmax: read S^T, mask, P^T = 2^(s - m) in bf16 into shared memory in the UMMA
//                     layout.  m is a per-row reference point (the score of the unit's first key), not
//                     the running maximum: the result is exact for any reference as long as nothing
//                     overflows, so the common tile needs no cross-thread reduction.  The four warps
//                     vote through a split-phase mbarrier on whether a score outgrew its reference by
//                     2^24 while the weights are already being formed; only then (rare) the references
//                     are raised, O^T is rescaled in TMEM and the tile is redone.  Row sums are kept per
//                     thread and left on the thread's TMEM lane at the end of the unit.
//   warps 4-7         epilogue: add the 128 lanes' row-sum shares up, O^T / sum out of one of two TMEM
//                     accumulator sets into the output or the split-KV partial; the last CTA of a
//                     (request, head) merges.  Runs beside the next unit's main loop.
// Every mbarrier wait is bounded; on expiry the CTA raises an abort flag, all roles leave their
// loops, STATUS_TIMEOUT is recorded, TMEM is freed and the kernel returns.  The softmax warps
// rendezvous on mbarriers (bounded), never on named barriers, so an aborting CTA cannot hang.
#include <cuda.h>
#include <cuda_bf16.h>

#include "nsd_internal.h"

namespace nsd {
namespace {

constexpr int kTileKeys = 128;
constexpr int kBlockSizeU = 16;                         // keys per pool block
constexpr int kBlocksPerTile = 8;
constexpr int kHalfBytes = kTileKeys * 128;              // [128 keys][64 dims] bf16 = 16 KiB
constexpr int kStageBytes = 2 * kHalfBytes;              // one K or one V tile: dims 0-63, dims 64-127
constexpr int kSoftmaxThreads = 128;                     // warps 0-3
constexpr int kEpilogueThreads = 128;                    // warps 4-7
constexpr int kWarpK = 8, kWarpV = 9, kWarpS = 10, kWarpPV = 11, kWarpQ = 12;
constexpr int kThreads = 13 * 32;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kMaxSlack = 24.0f;                       // a score may exceed its row's reference by 2^24
constexpr uint32_t kSpinLimit = 1u << 20;          // wait slices of ~2 us each

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
// Bounded wait.  try_wait parks the thread in hardware until the phase completes or a time slice (hinted at
// ~2 us) runs out, so waiting threads do not flood shared memory with polls; the slices are counted, and the
// wait gives up when the CTA's abort flag is raised or the budget (a few seconds) is spent.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    for (uint32_t i = 0; i < kSpinLimit; ++i) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(bar), "r"(parity), "r"(2000u)
            : "memory");
        if (done) return true;
#ifdef NSD_UMMA_BACKOFF
        __nanosleep(NSD_UMMA_BACKOFF);
#endif
        if (*abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}
#ifdef NSD_UMMA_PROF
// Development aid: per-role wait and section times of CTA 0, kept in registers and flushed once at the end.
__device__ long long g_prof[64];
__device__ __forceinline__ bool mbar_wait_p(uint32_t bar, uint32_t parity, volatile int* abort_flag, long long& acc, bool rec) {
    const long long t0 = clock64();
    const bool r = mbar_wait(bar, parity, abort_flag);
    if (rec) acc += clock64() - t0;
    return r;
}
#define PROF_DECL() long long prof_acc[32] = {0}
#define PROF_FLUSH() do { if (blockIdx.x == 0) { _Pragma("unroll") for (int i_ = 0; i_ < 32; ++i_) if (prof_acc[i_]) atomicAdd(reinterpret_cast<unsigned long long*>(&g_prof[i_]), (unsigned long long)prof_acc[i_]); } } while (0)
#define MBAR_WAIT(bar, par, ab, slot, rec) mbar_wait_p(bar, par, ab, prof_acc[slot], rec)
#define PROF_NOW() clock64()
#define PROF_ACC(slot, t0, rec) do { if (rec) prof_acc[slot] += clock64() - (t0); } while (0)
#define PROF_INC(slot, rec) do { if (rec) prof_acc[slot] += 1; } while (0)
#else
#define PROF_DECL() do {} while (0)
#define PROF_FLUSH() do {} while (0)
#define MBAR_WAIT(bar, par, ab, slot, rec) mbar_wait(bar, par, ab)
#define PROF_NOW() 0ll
#define PROF_ACC(slot, t0, rec) do { (void)(t0); } while (0)
#define PROF_INC(slot, rec) do {} while (0)
#endif
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// Named barriers of the two 128-thread groups: id 1 = softmax warps, id 2 = epilogue warps.
template <int ID>
__device__ __forceinline__ void group_bar_sync() { asm volatile("bar.sync %0, 128;" ::"n"(ID) : "memory"); }
template <int ID>
__device__ __forceinline__ bool group_bar_or(bool pred) {
    uint32_t out;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %1, 0;\n\tbarrier.red.or.pred p, %2, 128, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(out)
        : "r"((uint32_t)pred), "n"(ID)
        : "memory");
    return out != 0;
}

// Bounded rendezvous of the four softmax warps on an mbarrier (one arrival per warp); false once the CTA is aborting.
// The result is the same for every lane of a warp.
__device__ __forceinline__ bool group_sync(uint32_t bar, uint32_t& phase, int lane, volatile int* abort_flag) {
    __syncwarp();
    if (lane == 0) mbar_arrive(bar);
    const bool ok = mbar_wait(bar, phase & 1, abort_flag);
    ++phase;
    return !__any_sync(0xffffffffu, !ok);
}

// ---- TMA -----------------------------------------------------------------------------------------
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int32_t x, int32_t y, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
                 : "memory");
}

// ---- tcgen05 ---------------------------------------------------------------------------------------
// Shared-memory matrix descriptor: start address, leading / stride byte offsets (16-byte units),
// descriptor version 1, layout type (0 = no swizzle, 2 = 128-byte swizzle).
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t layout) {
    return (uint64_t)((saddr >> 4) & 0x3FFF) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16) |
           ((uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32) | ((uint64_t)1 << 46) | ((uint64_t)(layout & 7) << 61);
}
// Instruction descriptor, kind::f16: fp32 accumulate, bf16 A and B, majorness bits, N >> 3, M >> 4.
__device__ __forceinline__ uint32_t instr_desc(int M, int N, int a_mn_major, int b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn_major << 15) | ((uint32_t)b_mn_major << 16) |
           ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 16 consecutive columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16]) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const float (&v)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
        ::"r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])),
        "r"(__float_as_uint(v[3])), "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])),
        "r"(__float_as_uint(v[7])), "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])),
        "r"(__float_as_uint(v[11])), "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])),
        "r"(__float_as_uint(v[15]))
        : "memory");
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}

// Shared-memory and TMEM carve-up for R query-row columns.
template <int R>
struct Layout {
    static constexpr int kKStages = R <= 32 ? 3 : 2;
    static constexpr int kVStages = 3;
    static constexpr int kQHalfBytes = R * 128;                      // [R rows][64 dims]
    static constexpr int kQBytes = 2 * kQHalfBytes;
    static constexpr int kPBytes = kTileKeys * R * 2;                // P^T, bf16
    static constexpr int kPLbo = (R / 8) * 128;                      // next 8 keys
    static constexpr int kOffK = 0;
    static constexpr int kOffV = kOffK + kKStages * kStageBytes;
    static constexpr int kOffQ = kOffV + kVStages * kStageBytes;     // two buffers
    static constexpr int kOffP = kOffQ + 2 * kQBytes;                // two buffers
    static constexpr int kOffRed = kOffP + 2 * kPBytes;              // [4 warps][R] floats: tile maxima of a refresh
    static constexpr int kOffRedE = kOffRed + 4 * R * 4;             // [4 warps][R] floats: the epilogue's row-sum reduction
    static constexpr int kOffMref = kOffRedE + 4 * R * 4;            // [2][R] floats: minus the rows' reference points
    static constexpr int kOffBars = kOffMref + 2 * R * 4;            // 40 mbarrier slots, then five words
    static constexpr int kBytes = kOffBars + 40 * 8 + 32;
    // TMEM columns: three S^T buffers, two O^T accumulators, two sets of per-key row-sum shares.
    static constexpr int kTmemStride = R <= 32 ? 32 : 64;
    static constexpr int kTmemCols = R <= 32 ? 256 : 512;
    static constexpr int kTmemS = 0, kTmemO = 3 * kTmemStride, kTmemL = 5 * kTmemStride;
};
static_assert(Layout<32>::kBytes <= 227 * 1024 && Layout<48>::kBytes <= 227 * 1024 && Layout<64>::kBytes <= 227 * 1024,
              "shared memory budget");

}  // namespace
}  // namespace nsd

#include "verify_attn_umma_kernel.inc"

namespace nsd {

cudaError_t attn_umma_init() {
    cudaError_t e;
    if ((e = cudaFuncSetAttribute(verify_attn_umma_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, Layout<32>::kBytes)) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(verify_attn_umma_kernel<48>, cudaFuncAttributeMaxDynamicSharedMemorySize, Layout<48>::kBytes)) != cudaSuccess) return e;
    return cudaFuncSetAttribute(verify_attn_umma_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, Layout<64>::kBytes);
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

}  // namespace nsd

#ifdef NSD_UMMA_PROF
extern "C" void nsd_debug_umma_prof(long long* out, int reset) {
    cudaDeviceSynchronize();
    cudaMemcpyFromSymbol(out, nsd::g_prof, sizeof(long long) * 64);
    if (reset) {
        long long z[64] = {0};
        cudaMemcpyToSymbol(nsd::g_prof, z, sizeof(z));
    }
}
#endif
