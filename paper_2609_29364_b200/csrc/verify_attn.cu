// Verification attention: gamma+1 causal query rows per request over a paged,
// ragged KV cache with grouped-query heads (Appendix G.2: the target processes
// the anchor token plus the proposal tokens in one pass; Section 3: the KV state
// spans non-contiguous blocks addressed through a block map).
//
// Shape of the work.  For one request and one kv head, the (gamma+1) rows of the
// G = Hq/Hkv query heads that share the kv head are stacked into one M x D tile
// (M = G*(gamma+1) = 20 at gamma 4), so every K/V byte is read from HBM once and
// feeds all M rows through the tensor cores.  The arithmetic intensity is only
// ~20-36 flop per KV byte, so the kernel is bound by HBM bandwidth; the tensor
// cores (mma.sync m16n8k16, bf16 in / fp32 accumulate) keep the math off the
// critical path.
//
// Parallelisation (split-KV).  The host plan cuts each request's block range into
// chunks and orders (chunk) items longest first; the grid is one CTA per
// (item, kv head), scheduled by the hardware in that order.  A CTA has one warp
// per 16-row m-tile.  K/V tiles of 32 keys stream global -> shared through a
// cp.async ring (16-byte pieces, XOR-swizzled so ldmatrix is conflict free).
// Each warp keeps an online softmax (running max / sum in registers, quad
// shuffles) over its rows.  A request with one chunk writes bf16 output directly;
// otherwise the CTA stores its unnormalised fp32 partial (max, sum, acc) and the
// LAST CTA to finish that (request, head) -- decided by an atomic counter, no
// waiting -- merges all partials in chunk order and writes the output.
//
// Masking.  Row i sees keys [0, ctx + i].  Only tiles that reach past ctx need
// the mask.  Slots past ctx+gamma in the last block may hold anything (NaN
// included): scores there are replaced by -inf with a select, and the V rows of
// those slots are zeroed in shared memory, so 0 * NaN never reaches an
// accumulator.
#include <cuda_bf16.h>

#include <mutex>

#include "nsd_internal.h"

namespace nsd {
namespace {

constexpr int kBlockSize = 16;      // keys per pool block
constexpr int kTileKeys = 32;       // keys per pipeline stage (two pool blocks)
constexpr float kLog2e = 1.4426950408889634f;

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
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// Shared-memory tiles are [rows][D] bf16 with every row padded by 16 bytes: eight
// consecutive rows then start 16 bytes apart modulo 128, so the eight row reads of
// one ldmatrix phase hit distinct banks, and every address used in the main loop is
// "per-thread constant + compile-time offset" (no swizzle arithmetic per access).
template <int D>
struct Tile {
    static constexpr int kPitch = D * 2 + 16;                       // bytes per row
    static constexpr int kBytes = kTileKeys * kPitch;               // K (or V) of one stage
};

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <int D, int kStages>
struct Smem {
    static constexpr int kStageBytes = 2 * Tile<D>::kBytes;         // K then V
    static constexpr int kMaxChunkBlocks = 512;
    static constexpr int kBytes = kStages * kStageBytes + kMaxChunkBlocks * 4;
};

template <int D, int NMT, int kStages>
__global__ void __launch_bounds__(NMT * 32)
verify_attn_kernel(const AttnLaunch a) {
    constexpr int NT = NMT * 32;                  // threads
    constexpr int CPR = D / 8;                    // 16-byte pieces per row
    constexpr int KSTEPS = D / 16;                // k-steps of Q K^T
    constexpr int DT = D / 8;                     // n-tiles of P V
    constexpr int PITCH = Tile<D>::kPitch;
    constexpr int TILE = Tile<D>::kBytes;
    constexpr int STAGE = Smem<D, kStages>::kStageBytes;
    constexpr int ROWS_PER_STEP = NT / CPR;       // rows one pass of all threads covers in a block copy
    constexpr int COPY_STEPS = (kBlockSize + ROWS_PER_STEP - 1) / ROWS_PER_STEP;
    static_assert(NT % CPR == 0, "a copy pass covers whole rows");
    extern __shared__ __align__(128) unsigned char smem[];
    int32_t* blk_s = reinterpret_cast<int32_t*>(smem + kStages * STAGE);
    __shared__ int s_last;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int Hkv = a.shape.Hkv, Hq = a.shape.Hq, G = Hq / Hkv;
    const int item_idx = blockIdx.x / Hkv;
    const int head = blockIdx.x - item_idx * Hkv;
    const AttnItem it = a.items[item_idx];
    const int r = it.req;
    const int gamma = a.gamma;
    const int ctx = a.ctx_len[r];
    const int n_total = ctx + gamma + 1;          // keys that exist after the append
    const int M = a.m_rows;
    const int64_t table0 = a.kv_indptr[r];
    const int n_blk = it.blk_end - it.blk_begin;
    const int n_tiles = (n_blk + 1) >> 1;

    // ---- block ids of the chunk -> shared (bad ids are replaced by block 0 and reported)
    for (int i = tid; i < n_blk; i += NT) {
        int32_t b = a.kv_indices[table0 + it.blk_begin + i];
        if ((uint32_t)b >= (uint32_t)a.shape.num_blocks) {
            atomicOr(a.status, STATUS_BAD_BLOCK);
            atomicCAS(a.status + 1, 0, r + 1);
            b = 0;
        }
        blk_s[i] = b;
    }
    __syncthreads();                              // blk_s visible before tiles are issued

    // ---- per-thread constants of the copy and of the fragment loads
    const uint32_t smem0 = smem_u32(smem);
    const int cp_row = tid / CPR, cp_ch = tid - cp_row * CPR;
    const uint32_t cp_dst = smem0 + cp_row * PITCH + cp_ch * 16;               // + stage, K|V, half, step
    const int64_t block_elems = a.shape.block_elems();
    const uint16_t* k_src = a.pool_slab + (int64_t)head * (kBlockSize * D) + tid * 8;   // + block, step
    const int64_t v_off = (int64_t)Hkv * (kBlockSize * D);
    const int mi = lane >> 3;
    const uint32_t k_frag = smem0 + ((mi >> 1) * 8 + (lane & 7)) * PITCH + (mi & 1) * 16;          // + stage, half, kk
    const uint32_t v_frag = smem0 + TILE + ((mi & 1) * 8 + (lane & 7)) * PITCH + (mi >> 1) * 16;   // + stage, ks16, dp

    // Issues the copy of tile t (two pool blocks, K and V of this head) into `stage`.
    auto issue_tile = [&](int t, int stage) {
        if (t < n_tiles) {
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const int bi = 2 * t + half;
                const uint32_t dst = cp_dst + stage * STAGE + half * (kBlockSize * PITCH);
                if (bi < n_blk) {
                    const uint16_t* src = k_src + (int64_t)blk_s[bi] * block_elems;
#pragma unroll
                    for (int st = 0; st < COPY_STEPS; ++st) {
                        if ((st + 1) * ROWS_PER_STEP <= kBlockSize || cp_row + st * ROWS_PER_STEP < kBlockSize) {
                            cp_async16(dst + st * (ROWS_PER_STEP * PITCH), src + st * (NT * 8));
                            cp_async16(dst + TILE + st * (ROWS_PER_STEP * PITCH), src + v_off + st * (NT * 8));
                        }
                    }
                } else {                           // no such block: V must be finite (zero); K is masked
#pragma unroll
                    for (int st = 0; st < COPY_STEPS; ++st)
                        if (cp_row + st * ROWS_PER_STEP < kBlockSize)
                            *reinterpret_cast<int4*>(smem + (dst - smem0) + TILE + st * (ROWS_PER_STEP * PITCH)) = make_int4(0, 0, 0, 0);
                }
            }
        }
        cp_async_commit();
    };

#pragma unroll
    for (int s = 0; s < kStages - 1; ++s) issue_tile(s, s);

    // ---- per-warp state: rows g and g+8 of m-tile `warp`
    const int g = lane >> 2, tq = lane & 3;
    const int m_lo = warp * 16 + g, m_hi = m_lo + 8;
    const int lim_lo = ctx + min(m_lo / G, gamma);      // last visible key of the row
    const int lim_hi = ctx + min(m_hi / G, gamma);
    const float sc = rsqrtf((float)D) * kLog2e;          // raw score -> log2 domain
    float o_acc[DT][4];
#pragma unroll
    for (int i = 0; i < DT; ++i) o_acc[i][0] = o_acc[i][1] = o_acc[i][2] = o_acc[i][3] = 0.f;
    float mx_lo = -INFINITY, mx_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;
    // ---- Q fragments straight from global memory (row m = i*G + j is query row i of head head*G + j;
    //      rows past M are zero): a0/a2 = row g, a1/a3 = row g+8, columns kk*16 + {0,8} + 2*tq
    uint32_t qf[KSTEPS][4];
    {
        const uint16_t* q_lo = nullptr;
        const uint16_t* q_hi = nullptr;
        if (m_lo < M) q_lo = a.q + (((int64_t)r * (gamma + 1) + m_lo / G) * Hq + head * G + m_lo % G) * D + tq * 2;
        if (m_hi < M) q_hi = a.q + (((int64_t)r * (gamma + 1) + m_hi / G) * Hq + head * G + m_hi % G) * D + tq * 2;
#pragma unroll
        for (int kk = 0; kk < KSTEPS; ++kk) {
            qf[kk][0] = q_lo ? __ldg(reinterpret_cast<const uint32_t*>(q_lo + kk * 16)) : 0u;
            qf[kk][1] = q_hi ? __ldg(reinterpret_cast<const uint32_t*>(q_hi + kk * 16)) : 0u;
            qf[kk][2] = q_lo ? __ldg(reinterpret_cast<const uint32_t*>(q_lo + kk * 16 + 8)) : 0u;
            qf[kk][3] = q_hi ? __ldg(reinterpret_cast<const uint32_t*>(q_hi + kk * 16 + 8)) : 0u;
        }
    }

    const int key0_chunk = it.blk_begin * kBlockSize;
    // One tile: wait for its copy, refill the stage freed by the previous tile, S = Q K^T,
    // online softmax, O += P V.  `stage` is a compile-time constant at every call site.
    auto process_tile = [&](int t, int stage) {
        cp_async_wait<kStages - 2>();
        __syncthreads();
        issue_tile(t + kStages - 1, (stage + kStages - 1) % kStages);
        const int key0 = key0_chunk + t * kTileKeys;
        const bool need_mask = key0 + kTileKeys > ctx + 1;   // some key of the tile is hidden from some row
        if (key0 + kTileKeys > n_total) {                    // slots that hold no token: zero their V rows
            unsigned char* vs = smem + stage * STAGE + TILE;
            for (int c = tid; c < kTileKeys * CPR; c += NT) {
                const int row = c / CPR, ch = c - row * CPR;
                if (key0 + row >= n_total) *reinterpret_cast<int4*>(vs + row * PITCH + ch * 16) = make_int4(0, 0, 0, 0);
            }
            __syncthreads();
        }

        // ---- S = Q K^T (16 rows x 32 keys per warp)
        float s[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i) s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f;
#pragma unroll
        for (int kk = 0; kk < KSTEPS; ++kk) {
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                uint32_t kf[4];
                ldmatrix_x4(kf, k_frag + stage * STAGE + half * (16 * PITCH) + kk * 32);
                mma_bf16(s[half * 2 + 0], qf[kk], kf[0], kf[1]);
                mma_bf16(s[half * 2 + 1], qf[kk], kf[2], kf[3]);
            }
        }
        // ---- mask, online softmax (max over raw scores; the scale is folded into the exponent)
        float tmax_lo = -INFINITY, tmax_hi = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                if (need_mask) {
                    const int key = key0 + nt * 8 + tq * 2 + e;
                    s[nt][e] = key <= lim_lo ? s[nt][e] : -INFINITY;
                    s[nt][2 + e] = key <= lim_hi ? s[nt][2 + e] : -INFINITY;
                }
                tmax_lo = fmaxf(tmax_lo, s[nt][e]);
                tmax_hi = fmaxf(tmax_hi, s[nt][2 + e]);
            }
        }
        tmax_lo = fmaxf(tmax_lo, __shfl_xor_sync(0xffffffffu, tmax_lo, 1));
        tmax_lo = fmaxf(tmax_lo, __shfl_xor_sync(0xffffffffu, tmax_lo, 2));
        tmax_hi = fmaxf(tmax_hi, __shfl_xor_sync(0xffffffffu, tmax_hi, 1));
        tmax_hi = fmaxf(tmax_hi, __shfl_xor_sync(0xffffffffu, tmax_hi, 2));
        const float new_lo = fmaxf(mx_lo, tmax_lo), new_hi = fmaxf(mx_hi, tmax_hi);
        const bool grew = (new_lo != mx_lo) || (new_hi != mx_hi);
        const float off_lo = new_lo == -INFINITY ? 0.f : -new_lo * sc;   // nothing visible yet: avoid inf - inf
        const float off_hi = new_hi == -INFINITY ? 0.f : -new_hi * sc;
        if (__any_sync(0xffffffffu, grew)) {                // rescale only when some row's maximum moved
            const float resc_lo = ex2_approx(fmaf(mx_lo, sc, off_lo)), resc_hi = ex2_approx(fmaf(mx_hi, sc, off_hi));
            l_lo *= resc_lo;
            l_hi *= resc_hi;
#pragma unroll
            for (int i = 0; i < DT; ++i) {
                o_acc[i][0] *= resc_lo;
                o_acc[i][1] *= resc_lo;
                o_acc[i][2] *= resc_hi;
                o_acc[i][3] *= resc_hi;
            }
        }
        mx_lo = new_lo;
        mx_hi = new_hi;
        uint32_t pf[2][4];                               // P as A-fragments: [k-step of 16 keys]
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
            const float p0 = ex2_approx(fmaf(s[nt][0], sc, off_lo)), p1 = ex2_approx(fmaf(s[nt][1], sc, off_lo));
            const float p2 = ex2_approx(fmaf(s[nt][2], sc, off_hi)), p3 = ex2_approx(fmaf(s[nt][3], sc, off_hi));
            l_lo += p0 + p1;
            l_hi += p2 + p3;
            pf[nt >> 1][(nt & 1) * 2 + 0] = pack_bf16(p0, p1);
            pf[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16(p2, p3);
        }
        // ---- O += P V
#pragma unroll
        for (int ks16 = 0; ks16 < 2; ++ks16) {
#pragma unroll
            for (int dp = 0; dp < DT / 2; ++dp) {
                uint32_t vf[4];
                ldmatrix_x4_trans(vf, v_frag + stage * STAGE + ks16 * (16 * PITCH) + dp * 32);
                mma_bf16(o_acc[dp * 2 + 0], pf[ks16], vf[0], vf[1]);
                mma_bf16(o_acc[dp * 2 + 1], pf[ks16], vf[2], vf[3]);
            }
        }
    };

    for (int t = 0; t < n_tiles; t += kStages) {
#pragma unroll
        for (int s = 0; s < kStages; ++s)
            if (t + s < n_tiles) process_tile(t + s, s);
    }
    cp_async_wait<0>();

    // ---- row sums across the quad
    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);

    const int64_t row_base = (int64_t)r * (gamma + 1);
    if (it.part_base < 0) {
        // ---- single chunk: normalise and write bf16
#pragma unroll
        for (int hl = 0; hl < 2; ++hl) {
            const int m = hl ? m_hi : m_lo;
            if (m >= M) continue;
            const float l = hl ? l_hi : l_lo;
            const float inv = 1.f / l;
            const int i = m / G, j = m - i * G;
            const int64_t orow = ((row_base + i) * Hq + head * G + j);
            uint16_t* op = a.o + orow * D;
#pragma unroll
            for (int dt = 0; dt < DT; ++dt)
                *reinterpret_cast<uint32_t*>(op + dt * 8 + tq * 2) =
                    pack_bf16(o_acc[dt][hl * 2 + 0] * inv, o_acc[dt][hl * 2 + 1] * inv);
            if (a.lse && tq == 0) a.lse[orow] = ((hl ? mx_hi : mx_lo) * sc + log2f(l)) * 0.6931471805599453f;
        }
        return;
    }

    // ---- several chunks: store the partial, the last CTA of this (request, head) merges
    {
        const int64_t slot = ((int64_t)it.part_base + it.chunk_idx) * Hkv + head;
        float* pa = a.part_acc + slot * M * D;
        float* pm = a.part_ml + slot * M * 2;
#pragma unroll
        for (int hl = 0; hl < 2; ++hl) {
            const int m = hl ? m_hi : m_lo;
            if (m >= M) continue;
#pragma unroll
            for (int dt = 0; dt < DT; ++dt)
                *reinterpret_cast<float2*>(pa + (int64_t)m * D + dt * 8 + tq * 2) =
                    make_float2(o_acc[dt][hl * 2 + 0], o_acc[dt][hl * 2 + 1]);
            if (tq == 0) *reinterpret_cast<float2*>(pm + m * 2) = make_float2((hl ? mx_hi : mx_lo) * sc, hl ? l_hi : l_lo);
        }
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
    for (int e = tid; e < M * (D / 4); e += NT) {
        const int m = e / (D / 4), d4 = e - m * (D / 4);
        float mstar = -INFINITY;
        for (int c = 0; c < it.nchunks; ++c) {
            const int64_t slot = ((int64_t)it.part_base + c) * Hkv + head;
            mstar = fmaxf(mstar, __ldcg(a.part_ml + (slot * M + m) * 2));
        }
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        float l = 0.f;
        for (int c = 0; c < it.nchunks; ++c) {
            const int64_t slot = ((int64_t)it.part_base + c) * Hkv + head;
            const float2 ml = __ldcg(reinterpret_cast<const float2*>(a.part_ml + (slot * M + m) * 2));
            const float w = ml.x == -INFINITY ? 0.f : exp2f(ml.x - mstar);
            const float4 v = __ldcg(reinterpret_cast<const float4*>(a.part_acc + (slot * M + m) * D) + d4);
            acc.x += w * v.x;
            acc.y += w * v.y;
            acc.z += w * v.z;
            acc.w += w * v.w;
            l += w * ml.y;
        }
        const float inv = 1.f / l;
        const int i = m / G, j = m - i * G;
        const int64_t orow = ((row_base + i) * Hq + head * G + j);
        uint2 packed;
        packed.x = pack_bf16(acc.x * inv, acc.y * inv);
        packed.y = pack_bf16(acc.z * inv, acc.w * inv);
        *reinterpret_cast<uint2*>(a.o + orow * D + d4 * 4) = packed;
        if (a.lse && d4 == 0) a.lse[orow] = (mstar + log2f(l)) * 0.6931471805599453f;
    }
}

template <int D, int NMT, int kStages>
cudaError_t launch_one(const AttnLaunch& a, cudaStream_t stream) {
    const int64_t grid = (int64_t)a.n_items * a.shape.Hkv;
    verify_attn_kernel<D, NMT, kStages><<<(unsigned)grid, NMT * 32, Smem<D, kStages>::kBytes, stream>>>(a);
    return cudaGetLastError();
}

template <int D, int NMT, int kStages>
cudaError_t init_one() {
    return cudaFuncSetAttribute(verify_attn_kernel<D, NMT, kStages>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                Smem<D, kStages>::kBytes);
}

constexpr int kStagesD64 = 4, kStagesD128 = 3;

}  // namespace

cudaError_t attn_init() {
    cudaError_t e;
#define NSD_INIT(DD, NN, SS) \
    if ((e = init_one<DD, NN, SS>()) != cudaSuccess) return e;
    NSD_INIT(64, 1, kStagesD64) NSD_INIT(64, 2, kStagesD64) NSD_INIT(64, 3, kStagesD64) NSD_INIT(64, 4, kStagesD64)
    NSD_INIT(128, 1, kStagesD128) NSD_INIT(128, 2, kStagesD128) NSD_INIT(128, 3, kStagesD128) NSD_INIT(128, 4, kStagesD128)
    NSD_INIT(128, 2, 2) NSD_INIT(128, 2, 4)
#undef NSD_INIT
    return cudaSuccess;
}

cudaError_t launch_attn(const AttnLaunch& a, cudaStream_t stream) {
    if (a.n_items <= 0) return cudaSuccess;
    const int nmt = (a.m_rows + 15) / 16;
    if (a.shape.D == 128 && nmt == 2 && a.tune_stages == 2) return launch_one<128, 2, 2>(a, stream);
    if (a.shape.D == 128 && nmt == 2 && a.tune_stages == 4) return launch_one<128, 2, 4>(a, stream);
#define NSD_CASE(DD, NN, SS) \
    if (a.shape.D == DD && nmt == NN) return launch_one<DD, NN, SS>(a, stream);
    NSD_CASE(64, 1, kStagesD64) NSD_CASE(64, 2, kStagesD64) NSD_CASE(64, 3, kStagesD64) NSD_CASE(64, 4, kStagesD64)
    NSD_CASE(128, 1, kStagesD128) NSD_CASE(128, 2, kStagesD128) NSD_CASE(128, 3, kStagesD128) NSD_CASE(128, 4, kStagesD128)
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
            items[n_items++] = it;
        }
        if (n > 1) slots += (int)n;
    }

    int device = 0;
    if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= kMaxDevices) return NSD_ERR_CUDA;
    if (static_setup(device) != cudaSuccess) return NSD_ERR_CUDA;
    unsigned char* base = g_static_ptr[device];
    cudaStream_t st = static_cast<cudaStream_t>(stream);
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
    a.tune_stages = 0;
    return launch_attn(a, st) == cudaSuccess ? NSD_OK : NSD_ERR_CUDA;
}
