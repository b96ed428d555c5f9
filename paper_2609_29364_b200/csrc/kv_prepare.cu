// KV-state preparation: whole-block gather between pool regions and the append
// of the round's new tokens (Section 3, "KV cache organization": block-map
// traversal + fragmented copies, append-dominant state; Appendix E.2: the
// destination bank is filled before it computes).
//
// Both kernels only move bytes.  The gather moves contiguous (slab, block)
// chunks (64 KiB at the Qwen3-8B shape) with 32-byte accesses that bypass L1 and
// are marked evict-first, so a copy running beside attention does not push
// attention's tiles out of L2.
#include "nsd_internal.h"

namespace nsd {
namespace {

struct __align__(32) Vec32 {
    uint32_t w[8];
};
// 32-byte accesses (sm_100): no L1 allocation, evict-first in L2.
__device__ __forceinline__ Vec32 ld_stream(const void* p) {
    Vec32 v;
    asm volatile("ld.global.L1::no_allocate.L2::evict_first.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(v.w[0]), "=r"(v.w[1]), "=r"(v.w[2]), "=r"(v.w[3]), "=r"(v.w[4]), "=r"(v.w[5]), "=r"(v.w[6]), "=r"(v.w[7])
                 : "l"(p));
    return v;
}
__device__ __forceinline__ void st_stream(void* p, const Vec32& v) {
    asm volatile("st.global.L1::no_allocate.L2::evict_first.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p),
                 "r"(v.w[0]), "r"(v.w[1]), "r"(v.w[2]), "r"(v.w[3]), "r"(v.w[4]), "r"(v.w[5]), "r"(v.w[6]), "r"(v.w[7])
                 : "memory");
}

constexpr int kGatherThreads = 256;
constexpr int kGatherUnroll = 4;                                        // 32-byte accesses in flight per thread
constexpr int kGatherUnitBytes = kGatherThreads * kGatherUnroll * 32;   // 32 KiB per CTA iteration

// One unit = kGatherUnitBytes of one block pair.  block_bytes is a multiple of 32.
__global__ void __launch_bounds__(kGatherThreads)
gather_blocks_kernel(uint16_t* __restrict__ slab, int64_t n_pairs, const int32_t* __restrict__ src,
                     const int32_t* __restrict__ dst, int32_t num_blocks, int64_t block_bytes, int32_t units_per_block,
                     int32_t* __restrict__ status) {
    const int64_t n_units = n_pairs * units_per_block;
    for (int64_t u = blockIdx.x; u < n_units; u += gridDim.x) {
        const int64_t e = u / units_per_block;
        const int64_t off = (u - e * units_per_block) * (int64_t)kGatherUnitBytes;
        const int32_t s = __ldg(src + e), d = __ldg(dst + e);
        if ((uint32_t)s >= (uint32_t)num_blocks || (uint32_t)d >= (uint32_t)num_blocks) {
            if (threadIdx.x == 0) atomicOr(status, STATUS_BAD_BLOCK);
            continue;
        }
        const char* sp = reinterpret_cast<const char*>(slab) + (int64_t)s * block_bytes + off;
        char* dp = reinterpret_cast<char*>(slab) + (int64_t)d * block_bytes + off;
        const int64_t left = block_bytes - off;                     // bytes of this block still to copy
        Vec32 v[kGatherUnroll];
#pragma unroll
        for (int k = 0; k < kGatherUnroll; ++k) {
            const int64_t b = ((int64_t)k * kGatherThreads + threadIdx.x) * 32;
            if (b < left) v[k] = ld_stream(sp + b);
        }
#pragma unroll
        for (int k = 0; k < kGatherUnroll; ++k) {
            const int64_t b = ((int64_t)k * kGatherThreads + threadIdx.x) * 32;
            if (b < left) st_stream(dp + b, v[k]);
        }
    }
}

// One warp per (row, K|V): copies the Hkv head vectors of one new token into its slot.
__global__ void __launch_bounds__(256)
append_tokens_kernel(uint16_t* __restrict__ slab, Shape sh, int32_t batch, int32_t gamma,
                     const int32_t* __restrict__ ctx_len, const int64_t* __restrict__ kv_indptr,
                     const int32_t* __restrict__ kv_indices, const uint16_t* __restrict__ k_new,
                     const uint16_t* __restrict__ v_new, const uint8_t* __restrict__ is_migrated, int32_t subset,
                     int32_t* __restrict__ status) {
    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t n_rows = (int64_t)batch * (gamma + 1);
    if (warp >= 2 * n_rows) return;
    const int kv = (int)(warp & 1);
    const int64_t row = warp >> 1;
    const int r = (int)(row / (gamma + 1));
    const int t = (int)(row - (int64_t)r * (gamma + 1));
    if (subset != 0 && (int)(is_migrated[r] != 0) != (subset == 2)) return;
    const int64_t pos = (int64_t)ctx_len[r] + t;
    const int64_t entry = kv_indptr[r] + pos / sh.bs;
    const int slot = (int)(pos % sh.bs);
    int32_t b = -1;
    if (ctx_len[r] >= 0 && entry < kv_indptr[r + 1]) b = kv_indices[entry];
    if ((uint32_t)b >= (uint32_t)sh.num_blocks) {
        if (lane == 0) {
            atomicOr(status, STATUS_BAD_BLOCK);
            atomicCAS(status + 1, 0, r + 1);
        }
        return;
    }
    const uint16_t* srcv = (kv ? v_new : k_new) + row * sh.Hkv * sh.D;
    uint16_t* dstb = slab + (int64_t)b * sh.block_elems() + (int64_t)kv * sh.Hkv * sh.tile_elems() + (int64_t)slot * sh.D;
    const int vec_per_head = sh.D / 8;                              // 16-byte pieces per head vector
    const int n_vec = sh.Hkv * vec_per_head;
    for (int i = lane; i < n_vec; i += 32) {
        const int h = i / vec_per_head, c = i - h * vec_per_head;
        const int4 v = __ldg(reinterpret_cast<const int4*>(srcv + (int64_t)h * sh.D) + c);
        *(reinterpret_cast<int4*>(dstb + (int64_t)h * sh.tile_elems()) + c) = v;
    }
}

}  // namespace

cudaError_t launch_gather(const Shape& s, uint16_t* slab, int64_t n_pairs, const int32_t* src, const int32_t* dst,
                          int32_t* status, cudaStream_t stream) {
    if (n_pairs <= 0) return cudaSuccess;
    const int64_t block_bytes = s.block_elems() * 2;
    const int32_t upb = (int32_t)((block_bytes + kGatherUnitBytes - 1) / kGatherUnitBytes);
    const int64_t n_units = n_pairs * upb;
    // A bounded number of CTAs: the copy shares the SMs with attention.
    const int64_t max_ctas = 148 * 4;
    const int grid = (int)(n_units < max_ctas ? n_units : max_ctas);
    gather_blocks_kernel<<<grid, kGatherThreads, 0, stream>>>(slab, n_pairs, src, dst, s.num_blocks, block_bytes, upb, status);
    return cudaGetLastError();
}

cudaError_t launch_append(const Shape& s, uint16_t* slab, int32_t batch, int32_t gamma, const int32_t* ctx_len,
                          const int64_t* kv_indptr, const int32_t* kv_indices, const uint16_t* k_new,
                          const uint16_t* v_new, const uint8_t* is_migrated, int32_t subset, int32_t* status,
                          cudaStream_t stream) {
    const int64_t warps = 2LL * batch * (gamma + 1);
    if (warps <= 0) return cudaSuccess;
    const int grid = (int)((warps * 32 + 255) / 256);
    append_tokens_kernel<<<grid, 256, 0, stream>>>(slab, s, batch, gamma, ctx_len, kv_indptr, kv_indices, k_new, v_new,
                                                   is_migrated, subset, status);
    return cudaGetLastError();
}

}  // namespace nsd
