// Verification attention: gamma+1 causal query rows per request over a paged,
// ragged KV cache with grouped-query heads (Appendix G.2: the target processes
// the anchor token plus the proposal tokens in one pass; Section 3: the KV state
// spans non-contiguous blocks addressed through a block map).
//
// Shape of the work.  For one request and one kv head, the (gamma+1) rows of the
// G = Hq/Hkv query heads that share the kv head are stacked into M = G*(gamma+1)
// rows (20 at gamma 4), so every K/V byte is read from HBM once and feeds all M
// rows.  The arithmetic intensity is only ~20-36 flop per KV byte: the kernel is
// bound by HBM bandwidth and, under sustained load, by board power, so the design
// goal is the fewest instructions and shared-memory reads per KV byte.
//
// Transposed formulation.  With so few query rows the keys, not the queries, take
// the 16-wide M dimension of mma.sync.m16n8k16 (bf16 in, fp32 accumulate):
//     S^T = K  Q^T   A = K tile (16 keys x 16 dims, ldmatrix), B = Q^T held in registers
//     O^T = V^T P^T  A = V^T tile (16 dims x 16 keys, ldmatrix.trans), B = P^T
// The query rows are the 8-wide N dimension, so M is padded to a multiple of 8 (24)
// rather than 16 (32), every K/V fragment is loaded from shared memory once and
// reused for all row tiles, and one warp serves up to 24 rows.  P^T becomes a B
// operand by transposing the packed 8x8 accumulator blocks with movmatrix.
//
// Parallelisation (split-KV).  The host plan cuts each request's block range into
// chunks and orders the chunk items longest first; the grid is one CTA per
// (item, kv head), scheduled by the hardware in that order.  A CTA has one warp per
// group of up to three 8-row tiles (one warp at gamma 4).  K/V tiles of one pool block
// stream global -> shared through a four-stage ring (every fragment address a per-thread
// constant plus a compile-time offset; the ring loop is unrolled by stage), fed in one of
// two ways.  Tensor copies (the default where the shape is bound by HBM, up to four row
// tiles): four cp.async.bulk.tensor boxes of 16 keys x 64 dims per tile, issued by four
// lanes, land in the 128-byte-swizzled layout and complete on the stage's mbarrier; the
// consumer spends one wait and five instructions per tile on the feed instead of sixteen
// cp.async per lane, which is worth 4-6 % under the power cap.  cp.async (five or six row
// tiles, head_dim 64, gather-through, the allocation-free entry): rows padded by 16 bytes
// for conflict-free ldmatrix.  A request with one chunk writes bf16
// output directly; otherwise the CTA stores its unnormalised fp32 partial (max, sum,
// acc) and the LAST CTA to finish that (request, head) -- decided by an atomic
// counter, nobody waits -- merges all partials in chunk order and writes the output.
//
// Online softmax.  Each thread keeps the running maximum of its rows in the log2
// domain with the 1/sqrt(d)*log2(e) scale folded into one FFMA per score.  The
// running maximum is refreshed (and the accumulators rescaled) only when some score
// exceeds it by more than 2^8; until then probabilities are simply up to 256 times
// larger, which fp32 sums and bf16 operands carry without loss, and the common tile
// needs no cross-lane reduction at all.  Row sums are reduced across lanes once, at
// the end.
//
// Masking.  Row i sees keys [0, ctx + i].  Only tiles that reach past ctx need the
// mask.  Slots past ctx+gamma in the last block may hold anything (NaN included):
// scores there are replaced by -inf with a select, and the V rows of those slots are
// zeroed in shared memory, so 0 * NaN never reaches an accumulator.
#include <cuda_bf16.h>

#include <mutex>

#include "nsd_internal.h"

namespace nsd {
namespace {

constexpr int kBlockSize = 16;      // keys per pool block
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kMaxSlack = 8.0f;   // the running maximum may lag the true one by this much (log2 units)

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// Transposes an 8x8 matrix of 16-bit elements held one 32-bit register per lane.
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t x) {
    uint32_t y;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(y) : "r"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// ---- TMA-fed variant: mbarrier and tensor-copy helpers --------------------------------------------
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Bounded: gives up after `limit` hardware wait slices (2^20 by default: seconds); the caller then records
// STATUS_TIMEOUT and leaves.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, uint32_t limit) {
    for (uint32_t i = 0; i < limit; ++i) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(bar), "r"(parity), "r"(2000u)
            : "memory");
        if (done) return true;
    }
    return false;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int32_t x, int32_t y, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
                 : "memory");
}
// One box back to global memory (a bulk group of the issuing thread); x, y as for the load, never negative.
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, int32_t x, int32_t y, uint32_t src) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];" ::"l"(map), "r"(x), "r"(y), "r"(src) : "memory");
}

// Shared-memory tiles are [rows][D] bf16 with every row padded by 16 bytes: eight
// consecutive rows then start 16 bytes apart modulo 128, so the eight row reads of
// one ldmatrix phase hit distinct banks.
template <int D, int TK>
struct Tile {
    static constexpr int kPitch = D * 2 + 16;                       // bytes per row
    static constexpr int kBytes = TK * kPitch;                      // K (or V) of one stage
};

// TK = keys per pipeline stage (one or two pool blocks), kStages = ring depth.  The TMA-fed variant keeps the
// tiles unpadded in the 128-byte-swizzled layout the tensor copy writes: [K lo | K hi | V lo | V hi], each
// [TK keys][64 dims].
template <int D, int TK, int kStages, int ROWS, bool TMA = false>
struct Smem {
    static constexpr int kStageBytes = TMA ? 2 * TK * D * 2 : 2 * Tile<D, TK>::kBytes;     // K then V
    static constexpr int kMaxChunkBlocks = 256;                     // ids to read from + ids to write to
    static constexpr int kOutPitch = D + 4;                         // floats per staged output row
    static constexpr int kOutBytes = (ROWS * kOutPitch + 2 * ROWS) * 4;   // output staging reuses the ring
    static constexpr int kRingBytes = kStages * kStageBytes > kOutBytes ? kStages * kStageBytes : (kOutBytes + 15) / 16 * 16;
    static constexpr int kBytes = kRingBytes + 2 * kMaxChunkBlocks * 4 + (TMA ? 1024 : 0);
};

// NW warps, each serving NTW tiles of 8 query rows; rows m >= M are zero padding.  TMA = the K/V tiles arrive by
// cp.async.bulk.tensor boxes (one warp, head_dim 128, one pool block per stage, no gather-through) instead of cp.async.
// FUSE (TMA-fed variant only; the cp.async variant decides at run time): compiled with the gather-through path.  A
// separate instantiation, because carrying the path unused cost the plain kernel 5 % (registers, instruction fetch).
template <int D, int NW, int NTW, int TK, int kStages, bool TMA = false, bool FUSE = false>
__global__ void __launch_bounds__(NW * 32, ((NW == 2 && NTW == 2) || (NW == 3 && NTW == 1)) ? 6 : 1)   // six CTAs per SM, as shared memory allows, also where registers would not
verify_attn_kernel(const __grid_constant__ AttnLaunch a) {
    static_assert(!TMA || (D == 128 && TK == 16), "the TMA-fed variant covers head_dim 128 with one pool block per stage");
    constexpr int KG = TK / 16;                   // 16-key groups (= pool blocks) per tile
    constexpr int NT = NW * 32;                   // threads
    constexpr int CPR = D / 8;                    // 16-byte pieces per row
    constexpr int KSTEPS = D / 16;                // k-steps of K Q^T
    constexpr int DM = D / 16;                    // 16-dim m-tiles of V^T P^T
    constexpr int PITCH = Tile<D, TK>::kPitch;
    constexpr int TILE = Tile<D, TK>::kBytes;
    constexpr int ROWS_PAD = NW * NTW * 8;        // query rows incl. padding
    using SM = Smem<D, TK, kStages, ROWS_PAD, TMA>;
    pdl_release_dependents();                     // the next kernel on the stream may set itself up beside this grid's last wave
    constexpr int STAGE = SM::kStageBytes;
    constexpr int OPITCH = SM::kOutPitch;
    constexpr int ROWS_PER_STEP = NT / CPR;       // rows one pass of all threads covers in a block copy
    constexpr int COPY_STEPS = (kBlockSize + ROWS_PER_STEP - 1) / ROWS_PER_STEP;
    static_assert(NT % CPR == 0, "a copy pass covers whole rows");
    extern __shared__ __align__(128) unsigned char smem_raw[];
    // the swizzled tiles of the TMA-fed variant must start on a 1024-byte boundary (its size carries the slack)
    unsigned char* const smem = TMA ? reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023) : smem_raw;
    int32_t* blk_s = reinterpret_cast<int32_t*>(smem + SM::kRingBytes);
    __shared__ int s_last;
    __shared__ __align__(8) uint64_t full_bar[kStages];      // TMA-fed variant: a stage's bytes have landed
    __shared__ volatile int s_timeout;                       // ... or never did

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int Hkv = a.shape.Hkv, Hq = a.shape.Hq, G = Hq / Hkv;
    const int item_idx = blockIdx.x / Hkv;
    const int head = blockIdx.x - item_idx * Hkv;
    const AttnItem it = a.items[item_idx];
    const int r = it.req;
    const int gamma = it.gamma;                   // the request's own draft depth
    const int ctx = it.ctx;                       // the plan's copy of ctx_len[r]: one dependent load less before the first tile
    const int n_total = ctx + gamma + 1;          // keys that exist after the append
    const int M = G * (gamma + 1);                // stacked rows of this item (<= the rows the launch is shaped for)
    const int MS = a.m_stride;                    // rows per partial slot
    const int64_t table0 = it.tbl_off >= 0 ? (int64_t)it.tbl_off : a.kv_indptr[r];
    // a plan checked the table's length on the host; without one (tbl_off < 0) entries past the request's own are not followed
    const int64_t table_end = it.tbl_off >= 0 ? INT64_MAX : a.kv_indptr[r + 1];
    const int n_blk = it.blk_end - it.blk_begin;
    const int n_tiles = (n_blk + KG - 1) / KG;

    // Gather-through: a reassigned request streams its committed KV from the source blocks and writes it,
    // with the new tokens, to its destination blocks on the way (uniform per CTA).
    const bool fused = (TMA ? FUSE : a.fuse != 0) && it.src_off >= 0;
    const int n_src = (ctx + kBlockSize - 1) / kBlockSize;       // blocks that hold committed KV
    int32_t* dst_s = blk_s + SM::kMaxChunkBlocks;

    // ---- block ids of the chunk -> shared (bad ids are replaced by block 0 and reported);
    //      blk_s = where a tile is read from (-1: nowhere, a fresh block), dst_s = where it is written to
    for (int i = tid; i < n_blk; i += NT) {
        int32_t b = table0 + it.blk_begin + i < table_end ? a.kv_indices[table0 + it.blk_begin + i] : -1;
        if ((uint32_t)b >= (uint32_t)a.shape.num_blocks) {
            atomicOr(a.status, STATUS_BAD_BLOCK);
            atomicCAS(a.status + 1, 0, r + 1);
            b = 0;
        }
        if (fused) {
            dst_s[i] = b;
            b = -1;
            if (it.blk_begin + i < n_src) {
                b = a.mig_src[(int64_t)it.src_off + it.blk_begin + i];
                if ((uint32_t)b >= (uint32_t)a.shape.num_blocks) {
                    atomicOr(a.status, STATUS_BAD_BLOCK);
                    atomicCAS(a.status + 1, 0, r + 1);
                    b = 0;
                }
            }
        }
        blk_s[i] = b;
    }
    if (TMA && tid == 0) {
        s_timeout = 0;
        for (int s = 0; s < kStages; ++s) mbar_init(smem_u32(&full_bar[s]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();                              // blk_s (and the barriers) visible before tiles are issued

    // ---- per-thread constants of the copy and of the fragment loads
    const uint32_t smem0 = smem_u32(smem);
    const int cp_row = tid / CPR, cp_ch = tid - cp_row * CPR;
    const uint32_t cp_dst = smem0 + cp_row * PITCH + cp_ch * 16;               // + stage, K|V, half, step
    const int64_t block_elems = a.shape.block_elems();
    const uint16_t* k_src = a.pool_slab + (int64_t)head * (kBlockSize * D) + tid * 8;   // + block, step
    const int64_t v_off = (int64_t)Hkv * (kBlockSize * D);
    const int mi = lane >> 3;
    // K as A operand (16 keys x 16 dims): matrices (keys 0-7|8-15) x (dims 0-7|8-15) -> a0..a3
    const uint32_t k_frag = smem0 + ((mi & 1) * 8 + (lane & 7)) * PITCH + (mi >> 1) * 16;          // + stage, key group, kk
    // V^T as A operand (16 dims x 16 keys), read transposed: a0 = keys 0-7 x dims 0-7, a1 = keys 0-7 x dims 8-15,
    // a2 = keys 8-15 x dims 0-7, a3 = keys 8-15 x dims 8-15
    const uint32_t v_frag = smem0 + TILE + ((mi >> 1) * 8 + (lane & 7)) * PITCH + (mi & 1) * 16;   // + stage, key group, dm
    // TMA-fed variant: rows are 128 bytes and the 16-byte chunk c of row r sits at chunk c ^ (r & 7).  A fragment
    // load of k-step kk (or dim tile dm) reads chunk 2 * (kk & 3) + h of half kk >> 2, h = the lane's matrix column:
    // (2a + h) ^ x = 2a ^ (h ^ x), so four per-lane addresses cover every step with compile-time offsets on top.
    uint32_t k_sw[4], v_sw[4];
#pragma unroll
    for (int a2 = 0; a2 < 4; ++a2) {
        k_sw[a2] = smem0 + ((mi & 1) * 8 + (lane & 7)) * 128 + (((2 * a2) ^ ((mi >> 1) ^ (lane & 7))) << 4);
        v_sw[a2] = smem0 + ((mi >> 1) * 8 + (lane & 7)) * 128 + (((2 * a2) ^ ((mi & 1) ^ (lane & 7))) << 4);
    }

    // Issues the copy of tile t (KG pool blocks, K and V of this head) into `stage`.
    auto issue_tile = [&](int t, int stage) {
        if constexpr (TMA) {
            // four boxes of 16 keys x 64 dims (K lo, K hi, V lo, V hi), one per lane, completing on the stage's barrier
            if (t < n_tiles && warp == 0) {
                const uint32_t bar = smem_u32(&full_bar[stage]);
                // gather-through: the stage's previous tile may still be on its way out to its destination block
                if (fused && lane < 4) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                if (blk_s[t] >= 0) {
                    if (lane == 0) mbar_expect_tx(bar, STAGE);
                    __syncwarp();
                    if (lane < 4) {
                        const int32_t row = ((blk_s[t] * 2 + (lane >> 1)) * Hkv + head) * kBlockSize;
                        tma_load_2d(smem0 + stage * STAGE + lane * 2048, &a.tmap, (lane & 1) * 64, row, bar);
                    }
                } else {
                    // a fresh block (gather-through only): nothing to read.  V must be finite (zero); K is masked or injected.
                    __syncwarp();
                    for (int c = lane; c < 256; c += 32) *reinterpret_cast<int4*>(smem + stage * STAGE + 4096 + c * 16) = make_int4(0, 0, 0, 0);
                    __syncwarp();
                    if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
                }
            }
            return;
        }
        if (t < n_tiles) {
#pragma unroll
            for (int half = 0; half < KG; ++half) {
                const int bi = KG * t + half;
                const uint32_t dst = cp_dst + stage * STAGE + half * (kBlockSize * PITCH);
                if (bi < n_blk && blk_s[bi] >= 0) {
                    const uint16_t* src = k_src + (int64_t)blk_s[bi] * block_elems;
#pragma unroll
                    for (int st = 0; st < COPY_STEPS; ++st) {
                        if ((st + 1) * ROWS_PER_STEP <= kBlockSize || cp_row + st * ROWS_PER_STEP < kBlockSize) {
                            cp_async16(dst + st * (ROWS_PER_STEP * PITCH), src + st * (NT * 8));
                            cp_async16(dst + TILE + st * (ROWS_PER_STEP * PITCH), src + v_off + st * (NT * 8));
                        }
                    }
                } else {                           // nothing to read: V must be finite (zero); K is masked or injected
#pragma unroll
                    for (int st = 0; st < COPY_STEPS; ++st)
                        if (cp_row + st * ROWS_PER_STEP < kBlockSize)
                            *reinterpret_cast<int4*>(smem + (dst - smem0) + TILE + st * (ROWS_PER_STEP * PITCH)) = make_int4(0, 0, 0, 0);
                }
            }
        }
        cp_async_commit();
    };

    // Up to here the CTA has read its own inputs only (work item, block table) and set up shared memory; from here on it
    // reads the pool, which the kernel before this one on the stream (the append, a copy) writes.
    pdl_wait();
#pragma unroll
    for (int s = 0; s < kStages - 1; ++s) issue_tile(s, s);

    // ---- per-thread view of the fragments: keys g, g+8 of a 16-key group; rows 8j + 2tq + {0,1} of row tile j
    const int g = lane >> 2, tq = lane & 3;
    const int row0 = warp * (NTW * 8);                   // first query row of this warp
    const float sc = rsqrtf((float)D) * kLog2e;          // raw score -> log2 domain
    int lim[NTW][2];                                     // last visible key of each of the thread's rows
#pragma unroll
    for (int j = 0; j < NTW; ++j)
#pragma unroll
        for (int e = 0; e < 2; ++e) lim[j][e] = ctx + min((row0 + j * 8 + tq * 2 + e) / G, gamma);

    // ---- Q^T as B operand, straight from global memory: b0 = (dims 16kk + 2tq, +1; row g), b1 = dims + 8.
    //      Row m = i*G + h is query row i of head head*G + h; rows past M are zero.
    uint32_t qb[KSTEPS][NTW][2];
#pragma unroll
    for (int j = 0; j < NTW; ++j) {
        const int m = row0 + j * 8 + g;
        const uint16_t* qp = nullptr;
        if (m < M) qp = a.q + (((int64_t)it.row0 + m / G) * Hq + head * G + m % G) * D + tq * 2;
#pragma unroll
        for (int kk = 0; kk < KSTEPS; ++kk) {
            qb[kk][j][0] = qp ? __ldg(reinterpret_cast<const uint32_t*>(qp + kk * 16)) : 0u;
            qb[kk][j][1] = qp ? __ldg(reinterpret_cast<const uint32_t*>(qp + kk * 16 + 8)) : 0u;
        }
    }

    float oT[DM][NTW][4];                                // O^T: (dim 16dm + g, rows 2tq,2tq+1), (dim 16dm + g + 8, same rows)
#pragma unroll
    for (int dm = 0; dm < DM; ++dm)
#pragma unroll
        for (int j = 0; j < NTW; ++j) oT[dm][j][0] = oT[dm][j][1] = oT[dm][j][2] = oT[dm][j][3] = 0.f;
    float mrun[NTW][2], lsum[NTW][2];                    // running maximum (log2 domain) and this thread's share of the row sum
#pragma unroll
    for (int j = 0; j < NTW; ++j) mrun[j][0] = mrun[j][1] = -INFINITY, lsum[j][0] = lsum[j][1] = 0.f;

    const int key0_chunk = it.blk_begin * kBlockSize;
    // One tile: wait for its copy, refill the stage freed by the previous tile, S^T = K Q^T,
    // online softmax, O^T += V^T P^T.  `stage` is a compile-time constant at every call site.
    bool timed_out = false;                           // TMA-fed variant only: a stage never landed
    int t_failed = 0;
    const uint32_t wait_limit = a.wait_budget ? a.wait_budget : (1u << 20);
    auto process_tile = [&](int t, int stage) {
        if constexpr (TMA) {
            if (!mbar_wait(smem_u32(&full_bar[stage]), (uint32_t)((t / kStages) & 1), wait_limit)) s_timeout = 1;
            __syncthreads();                          // every thread is done with tile t - 1, whose stage is refilled next
            if (s_timeout) {                          // the same answer for every thread of the CTA
                timed_out = true;
                t_failed = t;
                return;
            }
        } else {
            cp_async_wait<kStages - 2>();
            __syncthreads();
        }
        issue_tile(t + kStages - 1, (stage + kStages - 1) % kStages);
        const int key0 = key0_chunk + t * TK;
        const bool need_mask = key0 + TK > ctx + 1;   // some key of the tile is hidden from some row
        if constexpr (TMA) {
            if (fused) {
                // Tiles sit as [K lo | K hi | V lo | V hi], each [16 keys][64 dims] with the 128-byte swizzle: the 16-byte
                // chunk c of row r of a part is at r * 128 + ((c ^ (r & 7)) << 4).
                unsigned char* ts = smem + stage * STAGE;
                const int p_lo = max(ctx, key0), p_hi = min(ctx + gamma, key0 + TK - 1);
                if (p_lo <= p_hi) {
                    // new tokens of this request that fall into the tile come from k_new / v_new, not from the pool
                    const int n_new = p_hi - p_lo + 1;
                    for (int c = tid; c < n_new * 32; c += NT) {
                        const int row = c >> 5, rem = c & 31, kv = rem >> 4, ch = rem & 15;
                        const int p = p_lo + row, rr = p - key0;
                        const uint16_t* nsrc = (kv ? a.v_new : a.k_new) + (((int64_t)it.row0 + (p - ctx)) * Hkv + head) * D + ch * 8;
                        *reinterpret_cast<int4*>(ts + (kv * 2 + (ch >> 3)) * 2048 + rr * 128 + (((ch & 7) ^ (rr & 7)) << 4)) =
                            __ldg(reinterpret_cast<const int4*>(nsrc));
                    }
                    __syncthreads();
                }
                if (blk_s[t] >= 0) {
                    // the whole tile goes to its destination block: four boxes, straight out of the stage
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncthreads();
                    if (warp == 0 && lane < 4) {
                        const int32_t row = ((dst_s[t] * 2 + (lane >> 1)) * Hkv + head) * kBlockSize;
                        tma_store_2d(&a.tmap, (lane & 1) * 64, row, smem0 + stage * STAGE + lane * 2048);
                        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                        // slots past the last token are about to be zeroed for the arithmetic: the copy must have read them
                        // first, because the destination block gets the source's tail slots verbatim
                        if (key0 + TK > n_total) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                    }
                    if (key0 + TK > n_total) __syncthreads();
                } else if (p_lo <= p_hi) {
                    // a fresh block: only the new tokens' rows are written, the other slots keep what they held
                    const int n_new = p_hi - p_lo + 1;
                    uint16_t* dbase = a.pool_slab_w + (int64_t)dst_s[t] * block_elems + (int64_t)head * (kBlockSize * D);
                    for (int c = tid; c < n_new * 32; c += NT) {
                        const int row = c >> 5, rem = c & 31, kv = rem >> 4, ch = rem & 15;
                        const int rr = p_lo + row - key0;
                        const int4 v = *reinterpret_cast<const int4*>(ts + (kv * 2 + (ch >> 3)) * 2048 + rr * 128 + (((ch & 7) ^ (rr & 7)) << 4));
                        *reinterpret_cast<int4*>(dbase + (int64_t)kv * v_off + rr * D + ch * 8) = v;
                    }
                }
            }
        } else if (fused) {
            unsigned char* ks = smem + stage * STAGE;
            // new tokens of this request that fall into the tile come from k_new / v_new, not from the pool
            const int p_lo = max(ctx, key0), p_hi = min(ctx + gamma, key0 + TK - 1);
            if (p_lo <= p_hi) {
                const int n_new = p_hi - p_lo + 1;
                for (int c = tid; c < n_new * 2 * CPR; c += NT) {
                    const int row = c / (2 * CPR), rem = c - row * (2 * CPR), kv = rem / CPR, ch = rem - kv * CPR;
                    const int p = p_lo + row;
                    const uint16_t* nsrc = (kv ? a.v_new : a.k_new) + (((int64_t)it.row0 + (p - ctx)) * Hkv + head) * D + ch * 8;
                    *reinterpret_cast<int4*>(ks + kv * TILE + (p - key0) * PITCH + ch * 16) = __ldg(reinterpret_cast<const int4*>(nsrc));
                }
                __syncthreads();
            }
            // write the tile to its destination blocks: whole blocks that had a source, else only the new tokens
#pragma unroll
            for (int half = 0; half < KG; ++half) {
                const int bi = KG * t + half;
                if (bi >= n_blk) continue;
                const bool whole = blk_s[bi] >= 0;
                const int r_lo = whole ? 0 : max(ctx - (key0 + half * 16), 0);
                const int r_hi = whole ? kBlockSize - 1 : min(ctx + gamma - (key0 + half * 16), kBlockSize - 1);
                uint16_t* dbase = a.pool_slab_w + (int64_t)dst_s[bi] * block_elems + (int64_t)head * (kBlockSize * D);
                for (int c = tid; c < (r_hi - r_lo + 1) * 2 * CPR; c += NT) {
                    const int row = r_lo + c / (2 * CPR), rem = c % (2 * CPR), kv = rem / CPR, ch = rem - kv * CPR;
                    const int4 v = *reinterpret_cast<const int4*>(ks + kv * TILE + (half * 16 + row) * PITCH + ch * 16);
                    *reinterpret_cast<int4*>(dbase + (int64_t)kv * v_off + row * D + ch * 8) = v;
                }
            }
            __syncthreads();                                  // the copy has read the tile before anything zeroes it
        }
        if (key0 + TK > n_total) {                    // slots that hold no token: zero their V rows
            if constexpr (TMA) {
                unsigned char* vs = smem + stage * STAGE + 4096;      // V lo, V hi: [16 keys][128 bytes] each
                for (int c = tid; c < TK * 16; c += NT) {
                    const int row = c >> 4, ch = c & 15;
                    if (key0 + row >= n_total) *reinterpret_cast<int4*>(vs + (ch >> 3) * 2048 + row * 128 + (ch & 7) * 16) = make_int4(0, 0, 0, 0);
                }
            } else {
                unsigned char* vs = smem + stage * STAGE + TILE;
                for (int c = tid; c < TK * CPR; c += NT) {
                    const int row = c / CPR, ch = c - row * CPR;
                    if (key0 + row >= n_total) *reinterpret_cast<int4*>(vs + row * PITCH + ch * 16) = make_int4(0, 0, 0, 0);
                }
            }
            __syncthreads();
        }

        // ---- S^T = K Q^T: KG groups of 16 keys x NTW row tiles
        float sT[KG][NTW][4];
#pragma unroll
        for (int kg = 0; kg < KG; ++kg)
#pragma unroll
            for (int j = 0; j < NTW; ++j) sT[kg][j][0] = sT[kg][j][1] = sT[kg][j][2] = sT[kg][j][3] = 0.f;
#pragma unroll
        for (int kk = 0; kk < KSTEPS; ++kk) {
#pragma unroll
            for (int kg = 0; kg < KG; ++kg) {
                uint32_t kf[4];
                if constexpr (TMA) ldmatrix_x4(kf, k_sw[kk & 3] + stage * STAGE + (kk >> 2) * 2048);
                else ldmatrix_x4(kf, k_frag + stage * STAGE + kg * (16 * PITCH) + kk * 32);
#pragma unroll
                for (int j = 0; j < NTW; ++j) mma_bf16(sT[kg][j], kf, qb[kk][j][0], qb[kk][j][1]);
            }
        }
        // ---- scale into the log2 domain, mask, thread-local maxima
        float tmax[NTW][2];
#pragma unroll
        for (int j = 0; j < NTW; ++j) tmax[j][0] = tmax[j][1] = -INFINITY;
#pragma unroll
        for (int kg = 0; kg < KG; ++kg)
#pragma unroll
            for (int j = 0; j < NTW; ++j)
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const int e = c & 1;
                    float v = sT[kg][j][c] * sc;
                    if (need_mask) {
                        const int key = key0 + kg * 16 + g + (c >> 1) * 8;
                        v = key <= lim[j][e] ? v : -INFINITY;
                    }
                    sT[kg][j][c] = v;
                    tmax[j][e] = fmaxf(tmax[j][e], v);
                }
        // ---- refresh the running maxima only when some score outgrows the slack
        bool outgrown = false;
#pragma unroll
        for (int j = 0; j < NTW; ++j)
#pragma unroll
            for (int e = 0; e < 2; ++e) outgrown |= tmax[j][e] > mrun[j][e] + kMaxSlack;
        if (__any_sync(0xffffffffu, outgrown)) {
#pragma unroll
            for (int j = 0; j < NTW; ++j)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    float v = tmax[j][e];                 // row maximum over the 8 lanes that share tq
                    v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 4));
                    v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 8));
                    v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 16));
                    const float m_new = fmaxf(mrun[j][e], v);
                    // nothing visible yet (m_new = -inf): keep everything at zero without forming inf - inf
                    const float resc = m_new == -INFINITY ? 1.f : ex2_approx(mrun[j][e] - m_new);
                    mrun[j][e] = m_new;
                    lsum[j][e] *= resc;
#pragma unroll
                    for (int dm = 0; dm < DM; ++dm) {
                        oT[dm][j][e] *= resc;
                        oT[dm][j][2 + e] *= resc;
                    }
                }
        }
        // ---- P^T = 2^(S^T - m) packed to bf16 and transposed into B fragments
        uint32_t pb[KG][NTW][2];
#pragma unroll
        for (int j = 0; j < NTW; ++j) {
            const float m0 = mrun[j][0] == -INFINITY ? 0.f : mrun[j][0];
            const float m1 = mrun[j][1] == -INFINITY ? 0.f : mrun[j][1];
#pragma unroll
            for (int kg = 0; kg < KG; ++kg) {
                const float p0 = ex2_approx(sT[kg][j][0] - m0), p1 = ex2_approx(sT[kg][j][1] - m1);   // key g
                const float p2 = ex2_approx(sT[kg][j][2] - m0), p3 = ex2_approx(sT[kg][j][3] - m1);   // key g + 8
                lsum[j][0] += p0 + p2;
                lsum[j][1] += p1 + p3;
                pb[kg][j][0] = movmatrix_trans(pack_bf16(p0, p1));
                pb[kg][j][1] = movmatrix_trans(pack_bf16(p2, p3));
            }
        }
        // ---- O^T += V^T P^T
#pragma unroll
        for (int kg = 0; kg < KG; ++kg) {
#pragma unroll
            for (int dm = 0; dm < DM; ++dm) {
                uint32_t vf[4];
                if constexpr (TMA) ldmatrix_x4_trans(vf, v_sw[dm & 3] + stage * STAGE + 4096 + (dm >> 2) * 2048);
                else ldmatrix_x4_trans(vf, v_frag + stage * STAGE + kg * (16 * PITCH) + dm * 32);
#pragma unroll
                for (int j = 0; j < NTW; ++j) mma_bf16(oT[dm][j], vf, pb[kg][j][0], pb[kg][j][1]);
            }
        }
    };

    for (int t = 0; t < n_tiles && !timed_out; t += kStages) {
#pragma unroll
        for (int s = 0; s < kStages; ++s)
            if (t + s < n_tiles && !timed_out) process_tile(t + s, s);
    }
    if (timed_out) {                                      // nothing is written for this item; the status word says why
        if (tid == 0) {
            atomicOr(a.status, STATUS_TIMEOUT);
            // the tiles armed after the one that never landed may still be arriving in this CTA's shared memory:
            // give each the same bounded wait before the memory goes back to the SM
            if constexpr (TMA) {
                for (int t2 = t_failed + 1; t2 < n_tiles && t2 < t_failed + kStages - 1; ++t2)
                    mbar_wait(smem_u32(&full_bar[t2 % kStages]), (uint32_t)((t2 / kStages) & 1), wait_limit);
            }
        }
        __syncthreads();
        return;
    }
    cp_async_wait<0>();
    if constexpr (TMA) {
        // gather-through: the last tiles may still be on their way out of the ring
        if (fused && warp == 0 && lane < 4) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    }
    __syncthreads();                                      // the ring is free: reuse it to stage the output

    // ---- row sums across the 8 lanes that share tq
#pragma unroll
    for (int j = 0; j < NTW; ++j)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            float v = lsum[j][e];
            v += __shfl_xor_sync(0xffffffffu, v, 4);
            v += __shfl_xor_sync(0xffffffffu, v, 8);
            v += __shfl_xor_sync(0xffffffffu, v, 16);
            lsum[j][e] = v;
        }
    // ---- stage O^T as [row][dim] fp32 (+ max, sum per row) so that the stores are row-contiguous
    float* out_s = reinterpret_cast<float*>(smem);
    float* ml_s = out_s + ROWS_PAD * OPITCH;              // [row][2]
#pragma unroll
    for (int j = 0; j < NTW; ++j)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const int m = row0 + j * 8 + tq * 2 + e;
#pragma unroll
            for (int dm = 0; dm < DM; ++dm) {
                out_s[m * OPITCH + dm * 16 + g] = oT[dm][j][e];
                out_s[m * OPITCH + dm * 16 + g + 8] = oT[dm][j][2 + e];
            }
            if (g == 0) {
                ml_s[m * 2] = mrun[j][e];
                ml_s[m * 2 + 1] = lsum[j][e];
            }
        }
    __syncthreads();

    const int64_t row_base = it.row0;
    if (it.part_base < 0) {
        // ---- single chunk: normalise and write bf16, 16 bytes per store
        for (int e = tid; e < M * (D / 8); e += NT) {
            const int m = e / (D / 8), d8 = e - m * (D / 8);
            const float inv = 1.f / ml_s[m * 2 + 1];
            const float4 x = *reinterpret_cast<const float4*>(out_s + m * OPITCH + d8 * 8);
            const float4 y = *reinterpret_cast<const float4*>(out_s + m * OPITCH + d8 * 8 + 4);
            const int i = m / G, h = m - i * G;
            const int64_t orow = (row_base + i) * Hq + head * G + h;
            uint4 packed;
            packed.x = pack_bf16(x.x * inv, x.y * inv);
            packed.y = pack_bf16(x.z * inv, x.w * inv);
            packed.z = pack_bf16(y.x * inv, y.y * inv);
            packed.w = pack_bf16(y.z * inv, y.w * inv);
            *reinterpret_cast<uint4*>(a.o + orow * D + d8 * 8) = packed;
            if (a.lse && d8 == 0) a.lse[orow] = (ml_s[m * 2] + log2f(ml_s[m * 2 + 1])) * 0.6931471805599453f;
        }
        return;
    }

    // ---- several chunks: store the partial, the last CTA of this (request, head) merges
    {
        const int64_t slot = ((int64_t)it.part_base + it.chunk_idx) * Hkv + head;
        float* pa = a.part_acc + slot * MS * D;
        float* pm = a.part_ml + slot * MS * 2;
        for (int e = tid; e < M * (D / 4); e += NT) {
            const int m = e / (D / 4), d4 = e - m * (D / 4);
            *reinterpret_cast<float4*>(pa + (int64_t)m * D + d4 * 4) = *reinterpret_cast<const float4*>(out_s + m * OPITCH + d4 * 4);
        }
        for (int e = tid; e < M * 2; e += NT) pm[e] = ml_s[e];
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        int32_t* cnt = a.counters + (int64_t)r * Hkv + head;
        const int old = atomicAdd(cnt, 1);
        const int last = (old == it.nchunks - 1);
        if (last) *cnt = 0;                               // ready for the next launch
        s_last = last;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    // Thread = one 4-dim column of RB rows at a time: the RB rows' loads of a chunk are independent, so a merge costs
    // about 2 * nchunks L2 round trips per row batch instead of per row.
    constexpr int C4 = D / 4, RP = NT / C4, RB = 8;
    static_assert(NT % C4 == 0, "threads cover whole rows of 4-dim columns");
    const int d4 = tid % C4;
    for (int mb = tid / C4; mb < M; mb += RP * RB) {
        float mstar[RB];
#pragma unroll
        for (int k = 0; k < RB; ++k) mstar[k] = -INFINITY;
        for (int c = 0; c < it.nchunks; ++c) {
            const float* ml = a.part_ml + (((int64_t)it.part_base + c) * Hkv + head) * MS * 2;
#pragma unroll
            for (int k = 0; k < RB; ++k) {
                const int m = mb + k * RP;
                if (m < M) mstar[k] = fmaxf(mstar[k], __ldcg(ml + m * 2));
            }
        }
        float4 acc[RB];
        float l[RB];
#pragma unroll
        for (int k = 0; k < RB; ++k) acc[k] = make_float4(0.f, 0.f, 0.f, 0.f), l[k] = 0.f;
        for (int c = 0; c < it.nchunks; ++c) {
            const int64_t slot = ((int64_t)it.part_base + c) * Hkv + head;
            float2 ml[RB];
            float4 v[RB];
#pragma unroll
            for (int k = 0; k < RB; ++k) {
                const int m = mb + k * RP;
                ml[k] = make_float2(-INFINITY, 0.f);
                v[k] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (m < M) {
                    ml[k] = __ldcg(reinterpret_cast<const float2*>(a.part_ml + (slot * MS + m) * 2));
                    v[k] = __ldcg(reinterpret_cast<const float4*>(a.part_acc + (slot * MS + m) * D) + d4);
                }
            }
#pragma unroll
            for (int k = 0; k < RB; ++k) {
                const float w = ml[k].x == -INFINITY ? 0.f : exp2f(ml[k].x - mstar[k]);
                acc[k].x += w * v[k].x;
                acc[k].y += w * v[k].y;
                acc[k].z += w * v[k].z;
                acc[k].w += w * v[k].w;
                l[k] += w * ml[k].y;
            }
        }
#pragma unroll
        for (int k = 0; k < RB; ++k) {
            const int m = mb + k * RP;
            if (m < M) {
                const float inv = 1.f / l[k];
                const int i = m / G, h = m - i * G;
                const int64_t orow = ((row_base + i) * Hq + head * G + h);
                uint2 packed;
                packed.x = pack_bf16(acc[k].x * inv, acc[k].y * inv);
                packed.y = pack_bf16(acc[k].z * inv, acc[k].w * inv);
                *reinterpret_cast<uint2*>(a.o + orow * D + d4 * 4) = packed;
                if (a.lse && d4 == 0) a.lse[orow] = (mstar[k] + log2f(l[k])) * 0.6931471805599453f;
            }
        }
    }
}

template <int D, int NW, int NTW, int TK, int kStages, bool TMA = false, bool FUSE = false>
cudaError_t launch_one(const AttnLaunch& a, cudaStream_t stream) {
    const int64_t grid = (int64_t)a.n_items * a.shape.Hkv;
    return launch_kernel(verify_attn_kernel<D, NW, NTW, TK, kStages, TMA, FUSE>, dim3((unsigned)grid), dim3(NW * 32),
                         Smem<D, TK, kStages, NW * NTW * 8, TMA>::kBytes, stream, a.pdl != 0, a);
}

template <int D, int NW, int NTW, int TK, int kStages, bool TMA = false, bool FUSE = false>
cudaError_t init_one() {
    return cudaFuncSetAttribute(verify_attn_kernel<D, NW, NTW, TK, kStages, TMA, FUSE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                Smem<D, TK, kStages, NW * NTW * 8, TMA>::kBytes);
}

// One pool block per stage and a deeper ring gave the most resident warps per SM at the same bytes in flight.
constexpr int kTileKeys = 16, kStagesD64 = 4, kStagesD128 = 4;

// Row tiles of 8: 1..8 of them, spread over warps of at most three tiles each; and two or three tiles over as many
// warps of one tile each, for grids that do not fill the machine.
#define NSD_ATTN_SHAPES(X, DD, SS) \
    X(DD, 1, 1, kTileKeys, SS) X(DD, 1, 2, kTileKeys, SS) X(DD, 1, 3, kTileKeys, SS) X(DD, 2, 2, kTileKeys, SS) X(DD, 2, 3, kTileKeys, SS) X(DD, 3, 3, kTileKeys, SS) \
    X(DD, 2, 1, kTileKeys, SS) X(DD, 3, 1, kTileKeys, SS)

}  // namespace

cudaError_t attn_init() {
    cudaError_t e;
#define NSD_INIT(DD, WW, TT, KK, SS) \
    if ((e = init_one<DD, WW, TT, KK, SS>()) != cudaSuccess) return e;
    NSD_ATTN_SHAPES(NSD_INIT, 64, kStagesD64)
    NSD_ATTN_SHAPES(NSD_INIT, 128, kStagesD128)
#define NSD_INIT_TMA(DD, WW, TT, KK, SS) \
    if ((e = init_one<DD, WW, TT, KK, SS, true>()) != cudaSuccess) return e; \
    if ((e = init_one<DD, WW, TT, KK, SS, true, true>()) != cudaSuccess) return e;
    NSD_ATTN_SHAPES(NSD_INIT_TMA, 128, kStagesD128)
#undef NSD_INIT_TMA
#undef NSD_INIT
    return cudaSuccess;
}

cudaError_t launch_attn(const AttnLaunch& a, cudaStream_t stream) {
    if (a.n_items <= 0) return cudaSuccess;
    const int nt8 = (a.m_rows + 7) / 8;                  // row tiles needed
    if (nt8 < 1 || nt8 > 8) return cudaErrorInvalidValue;
    int nw = (nt8 + 2) / 3, ntw = (nt8 + nw - 1) / nw;
    // A grid that fits the machine's CTA slots runs as one wave, and the wave lasts as long as one warp takes over its
    // longest item's tiles: HBM is not the limit there.  Two or three row tiles then go to as many warps of one tile.
    if (nw == 1 && ntw > 1 && a.cta_slots > 0 && (int64_t)a.n_items * a.shape.Hkv <= a.cta_slots) nw = ntw, ntw = 1;
    // K/V tiles by tensor copies where that measured faster: the shapes that are bound by HBM (up to 32 stacked rows:
    // +4-6 % at 20-24 rows, +3 % at 28-32).  The five- and six-row-tile shapes are bound by the tensor pipe and by
    // shared-memory reads and ran 8-25 % slower fed this way, so they stay on cp.async.
    if (a.tma_feed && a.tmap_valid && a.shape.D == 128 && (nw == 1 || ntw == 1 || (nw == 2 && ntw == 2))) {
#define NSD_TMA_CASE(DD, WW, TT, KK, SS) \
        if (nw == WW && ntw == TT) return a.fuse ? launch_one<DD, WW, TT, KK, SS, true, true>(a, stream) : launch_one<DD, WW, TT, KK, SS, true>(a, stream);
        NSD_ATTN_SHAPES(NSD_TMA_CASE, 128, kStagesD128)
#undef NSD_TMA_CASE
    }
#define NSD_CASE(DD, WW, TT, KK, SS) \
    if (a.shape.D == DD && nw == WW && ntw == TT) return launch_one<DD, WW, TT, KK, SS>(a, stream);
    NSD_ATTN_SHAPES(NSD_CASE, 64, kStagesD64)
    NSD_ATTN_SHAPES(NSD_CASE, 128, kStagesD128)
#undef NSD_CASE
    return cudaErrorInvalidValue;
}

}  // namespace nsd

// =====================================================================================
// nsd_verify_attn_static: the same attention kernel for callers that cannot allocate.
//
// Some hosts of this library may not call cudaMalloc at all: a plugin running inside
// another runtime's memory budget, a worker whose device memory was carved up once at
// start-up (the paper's pre-allocated KV banks are that kind of process), code on a
// latency path where an allocator call could block on a device-wide synchronisation.
// For them the split-KV scratch (work list, arrival counters, fp32 partials, status word)
// lives in the file-scope device array below instead of a caller workspace.  Every GPU
// that loads the library carries the array until the process exits, so it is kept small
// and the entry point refuses batches that do not fit.
// =====================================================================================
namespace nsd {
namespace {

constexpr int kStaticMaxBatch = 64;        // requests per call
constexpr int kStaticMaxSlots = 64;        // chunks of requests that were split (partials kept)
constexpr int kStaticMaxItems = kStaticMaxBatch + kStaticMaxSlots;
constexpr int kStaticMaxHkv = 8;
constexpr int kStaticMaxRows = 32;         // (Hq/Hkv) * (gamma+1)
constexpr int kStaticMaxD = 128;
constexpr int kStaticChunkBlocks = 64;     // 1024 keys per chunk

constexpr size_t kStaticOffStatus = 0;
constexpr size_t kStaticOffCounters = 256;
constexpr size_t kStaticOffItems = kStaticOffCounters + sizeof(int32_t) * kStaticMaxBatch * kStaticMaxHkv;
constexpr size_t kStaticOffMl = kStaticOffItems + sizeof(AttnItem) * kStaticMaxItems;
constexpr size_t kStaticOffAcc = kStaticOffMl + sizeof(float) * 2 * kStaticMaxSlots * kStaticMaxHkv * kStaticMaxRows;
constexpr size_t kStaticBytes = kStaticOffAcc + sizeof(float) * kStaticMaxSlots * kStaticMaxHkv * kStaticMaxRows * kStaticMaxD;
static_assert(kStaticOffItems % 256 == 0 && kStaticOffMl % 256 == 0 && kStaticOffAcc % 256 == 0, "scratch sections stay 256-byte aligned");
static_assert(kStaticBytes <= (9u << 20), "the static scratch is meant to stay modest (about 8.1 MiB)");

// In host code this name is only a handle for cudaGetSymbolAddress; it is NOT a device
// address and must never be handed to a kernel as a pointer.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

constexpr int kMaxDevices = 64;
unsigned char* g_static_ptr[kMaxDevices];   // device address of the array, per device, set once
bool g_static_ready[kMaxDevices];
std::mutex g_static_mutex;

// Once per device, with that device current: resolve the array's device address and opt
// the kernels in to their shared-memory size.  Neither call allocates.
cudaError_t static_setup(int device) {
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (g_static_ready[device]) return cudaSuccess;
    void* ptr = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
    if (e != cudaSuccess) return e;
    if (ptr == nullptr) return cudaErrorInvalidSymbol;
    if ((e = attn_init()) != cudaSuccess) return e;
    g_static_ptr[device] = static_cast<unsigned char*>(ptr);
    g_static_ready[device] = true;
    return cudaSuccess;
}

}  // namespace
}  // namespace nsd

extern "C" nsd_status nsd_verify_attn_static(const void* kv_slab, int32_t num_blocks, int32_t num_q_heads,
                                             int32_t num_kv_heads, int32_t head_dim, int32_t block_size,
                                             const void* q, void* o, int32_t batch, int32_t gamma,
                                             const int32_t* h_ctx_len, const int32_t* ctx_len,
                                             const int64_t* kv_indptr, const int32_t* kv_indices, void* stream) {
    using namespace nsd;
    if (batch < 0 || gamma < 1 || num_blocks < 1 || num_q_heads < 1 || num_kv_heads < 1) return NSD_ERR_INVALID_ARG;
    if (num_q_heads % num_kv_heads) return NSD_ERR_INVALID_ARG;
    if ((head_dim != 64 && head_dim != 128) || block_size != kBlockSize) return NSD_ERR_UNSUPPORTED;
    const int rows = (num_q_heads / num_kv_heads) * (gamma + 1);
    if (batch > kStaticMaxBatch || num_kv_heads > kStaticMaxHkv || rows > kStaticMaxRows) return NSD_ERR_CAPACITY;
    if (batch == 0) return NSD_OK;
    if (!kv_slab || !q || !o || !h_ctx_len || !ctx_len || !kv_indptr || !kv_indices) return NSD_ERR_INVALID_ARG;

    // work list on the stack: requests longer than one chunk are split and keep partials
    AttnItem items[kStaticMaxItems];
    int n_items = 0, slots = 0;
    for (int r = 0; r < batch; ++r) {
        if (h_ctx_len[r] < 0) return NSD_ERR_INVALID_ARG;
        const int64_t need = ((int64_t)h_ctx_len[r] + gamma + 1 + kBlockSize - 1) / kBlockSize;
        const int64_t n = (need + kStaticChunkBlocks - 1) / kStaticChunkBlocks;
        if (n_items + n > kStaticMaxItems || (n > 1 && slots + n > kStaticMaxSlots)) return NSD_ERR_CAPACITY;
        for (int c = 0; c < (int)n; ++c) {
            AttnItem it{};
            it.req = r;
            it.blk_begin = c * kStaticChunkBlocks;
            it.blk_end = (int32_t)(need < (int64_t)(c + 1) * kStaticChunkBlocks ? need : (int64_t)(c + 1) * kStaticChunkBlocks);
            it.part_base = n > 1 ? slots : -1;
            it.chunk_idx = c;
            it.nchunks = (int32_t)n;
            it.ctx = h_ctx_len[r];
            it.gamma = gamma;
            it.row0 = r * (gamma + 1);
            it.tbl_off = -1;                              // this entry point has no host copy of kv_indptr
            items[n_items++] = it;
        }
        if (n > 1) slots += (int)n;
    }

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // the work list below is uploaded from this stack frame: a captured copy node would outlive it
    cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &capturing) != cudaSuccess) return NSD_ERR_CUDA;
    if (capturing != cudaStreamCaptureStatusNone) return NSD_ERR_INVALID_ARG;
    int device = 0;
    if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= kMaxDevices) return NSD_ERR_CUDA;
    if (static_setup(device) != cudaSuccess) return NSD_ERR_CUDA;
    unsigned char* base = g_static_ptr[device];
    // The array keeps whatever the previous call left: status and counters must start at zero.
    if (cudaMemsetAsync(base, 0, kStaticOffItems, st) != cudaSuccess) return NSD_ERR_CUDA;
    // The source is pageable (this stack frame): the runtime has staged it when the call returns.
    if (cudaMemcpyAsync(base + kStaticOffItems, items, sizeof(AttnItem) * n_items, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return NSD_ERR_CUDA;

    AttnLaunch a{};
    a.shape = Shape{1, num_blocks, num_q_heads, num_kv_heads, head_dim, block_size};
    a.pool_slab = static_cast<const uint16_t*>(kv_slab);
    a.q = static_cast<const uint16_t*>(q);
    a.o = static_cast<uint16_t*>(o);
    a.lse = nullptr;
    a.ctx_len = ctx_len;
    a.kv_indptr = kv_indptr;
    a.kv_indices = kv_indices;
    a.items = reinterpret_cast<const AttnItem*>(base + kStaticOffItems);
    a.n_items = n_items;
    a.gamma = gamma;
    a.part_acc = reinterpret_cast<float*>(base + kStaticOffAcc);
    a.part_ml = reinterpret_cast<float*>(base + kStaticOffMl);
    a.counters = reinterpret_cast<int32_t*>(base + kStaticOffCounters);
    a.status = reinterpret_cast<int32_t*>(base + kStaticOffStatus);
    a.m_rows = rows;
    a.m_stride = rows;
    return launch_attn(a, st) == cudaSuccess ? NSD_OK : NSD_ERR_CUDA;
}
