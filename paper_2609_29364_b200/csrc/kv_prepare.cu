// KV-state preparation: whole-block gather between pool regions and the append
// of the round's new tokens (Section 3, "KV cache organization": block-map
// traversal + fragmented copies, append-dominant state; Appendix E.2: the
// destination bank is filled before it computes).
//
// Both kernels only move bytes.  The gather moves contiguous (slab, block)
// chunks (64 KiB at the Qwen3-8B shape) with bulk asynchronous copies
// (cp.async.bulk, the 1-D TMA path): global -> shared -> global, driven by one
// thread per CTA, so a copy running beside attention costs the SMs almost no
// issue slots.
#include "nsd_internal.h"

namespace nsd {
namespace {

// ---- gather: bulk copies (TMA) ------------------------------------------------------
// One elected thread per CTA moves kBulkBytes pieces global -> shared -> global with
// cp.async.bulk, kBulkSlots pieces in flight: the load of a piece completes on an
// mbarrier (transaction bytes), its store is a bulk group, and a slot is reused once the
// store has finished READING shared memory.  No other thread touches the data, so the SM
// spends a handful of instructions per 16 KiB.  Every wait is bounded: on a timeout the
// CTA records STATUS_TIMEOUT, waits (bounded again) for the loads it has armed, so that no
// copy lands in shared memory the CTA has given back, waits for its stores and returns.
constexpr int kBulkBytes = 16 * 1024;
constexpr int kBulkSlots = 4;
// A slot is refilled while up to kBulkBehind - 1 younger stores may still be reading shared memory, i.e. the loads run
// kBulkSlots - kBulkBehind pieces ahead.  Measured alone (10 272 block pairs): 1 -> 5.6 TB/s (every refill waits
// for the store issued just before it), 2 -> 6.1 TB/s.  Six slots in two CTAs per SM reach 6.45 TB/s alone but
// cost the fused round 1 % (96 KiB CTAs find room beside the attention CTAs less often), so the round keeps four.
constexpr int kBulkBehind = 2;
constexpr int kBulkCtasPerSm = 4;
constexpr uint32_t kBulkSpinLimit = 1u << 22;

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, uint32_t limit) {
    for (uint32_t i = 0; i < limit; ++i) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(bar), "r"(parity)
            : "memory");
        if (done) return true;
    }
    return false;
}

__global__ void __launch_bounds__(32)
gather_blocks_bulk_kernel(uint16_t* __restrict__ slab, int64_t n_pairs, const int32_t* __restrict__ src,
                          const int32_t* __restrict__ dst, int32_t num_blocks, int64_t block_bytes,
                          int32_t pieces_per_block, int32_t* __restrict__ status, uint32_t spin_limit,
                          uint32_t starve_bytes) {
    extern __shared__ __align__(128) unsigned char bulk_smem[];
    __shared__ __align__(8) uint64_t full_bar[kBulkSlots];
    pdl_release_dependents();                           // whatever follows on the stream may set itself up meanwhile
    if (threadIdx.x != 0) return;                       // a single thread drives the copy engine
    for (int s = 0; s < kBulkSlots; ++s)
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_addr(&full_bar[s])) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");

    const int64_t n_pieces = n_pairs * pieces_per_block;
    const int64_t first = blockIdx.x, stride = gridDim.x;
    const int64_t mine = first < n_pieces ? (n_pieces - first + stride - 1) / stride : 0;
    auto piece_ptrs = [&](int64_t k, const char*& sp, char*& dp, uint32_t& bytes) -> bool {
        const int64_t u = first + k * stride;
        const int64_t e = u / pieces_per_block;
        const int64_t off = (u - e * pieces_per_block) * (int64_t)kBulkBytes;
        const int32_t sb = __ldg(src + e), db = __ldg(dst + e);
        if ((uint32_t)sb >= (uint32_t)num_blocks || (uint32_t)db >= (uint32_t)num_blocks) {
            atomicOr(status, STATUS_BAD_BLOCK);
            return false;
        }
        sp = reinterpret_cast<const char*>(slab) + (int64_t)sb * block_bytes + off;
        dp = reinterpret_cast<char*>(slab) + (int64_t)db * block_bytes + off;
        const int64_t left = block_bytes - off;
        bytes = (uint32_t)(left < kBulkBytes ? left : kBulkBytes);
        return true;
    };
    auto issue_load = [&](int64_t k) {
        const int s = (int)(k % kBulkSlots);
        const char* sp; char* dp; uint32_t bytes;
        const uint32_t bar = smem_addr(&full_bar[s]);
        if (!piece_ptrs(k, sp, dp, bytes)) {            // nothing to copy: complete the phase by hand
            asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
            return;
        }
        // starve_bytes is zero outside the bounded-wait test, which makes the phase impossible to complete
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes + starve_bytes) : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(smem_addr(bulk_smem + s * kBulkBytes)), "l"(sp), "r"(bytes), "r"(bar) : "memory");
    };

    // Slot reuse: the load of piece k needs the store of piece k - kBulkSlots to have read its data.
    // Stores are committed one group per piece, in order, so "at most kBehind - 1 groups still reading" is the condition.
    constexpr int kBehind = kBulkBehind;
    constexpr int kAhead = kBulkSlots - kBehind;
    bool ok = true;
    int64_t issued = 0;                                 // loads armed so far: pieces [0, issued)
    for (; issued < kAhead && issued < mine; ++issued) issue_load(issued);
    int64_t k = 0;
    for (; k < mine; ++k) {
        if (issued < mine) {
            // the slot of piece `issued` = k + kAhead was last used by piece k - kBehind: that store must have finished reading
            asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(kBehind - 1) : "memory");
            issue_load(issued++);
        }
        const int s = (int)(k % kBulkSlots);
        ok = mbar_wait_bounded(smem_addr(&full_bar[s]), (uint32_t)((k / kBulkSlots) & 1), spin_limit);
        if (!ok) break;
        const char* sp; char* dp; uint32_t bytes;
        if (piece_ptrs(k, sp, dp, bytes)) {
            asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                         ::"l"(dp), "r"(smem_addr(bulk_smem + s * kBulkBytes)), "r"(bytes) : "memory");
        }
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    }
    if (!ok) {
        atomicOr(status, STATUS_TIMEOUT);
        // the loads armed after piece k may still be writing this CTA's shared memory: give each of them the same
        // bounded wait before the memory goes back to the SM
        for (int64_t j = k + 1; j < issued; ++j)
            mbar_wait_bounded(smem_addr(&full_bar[j % kBulkSlots]), (uint32_t)((j / kBulkSlots) & 1), spin_limit);
    }
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // all stores complete before the CTA retires
}

// One warp per (row, K|V): copies the Hkv head vectors of one new token into its slot.
__global__ void __launch_bounds__(256)
append_tokens_kernel(uint16_t* __restrict__ slab, Shape sh, int32_t batch, int32_t gamma,
                     const int64_t* __restrict__ q_indptr, const int32_t* __restrict__ ctx_len, const int64_t* __restrict__ kv_indptr,
                     const int32_t* __restrict__ kv_indices, const uint16_t* __restrict__ k_new,
                     const uint16_t* __restrict__ v_new, const uint8_t* __restrict__ is_migrated, int32_t subset,
                     int32_t* __restrict__ status) {
    // Everything up to the stores reads the call's own inputs only; the stores go into blocks that the kernel before
    // this one on the stream (a copy into the same blocks, or the attention of the layer that shares the slab) may
    // still be writing or reading.  Every thread passes the wait, also those with nothing to store: the grid must not
    // complete before its predecessor has, because the kernel after this one waits for this grid only.
    pdl_release_dependents();
    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t n_rows = (int64_t)batch * (gamma + 1);
    const uint16_t* srcv = nullptr;
    uint16_t* dstb = nullptr;
    [&]() {
        if (warp >= 2 * n_rows) return;
        const int kv = (int)(warp & 1);
        int64_t row = warp >> 1;                                    // (request, token) over the padded grid batch x (gamma + 1)
        const int r = (int)(row / (gamma + 1));
        const int t = (int)(row - (int64_t)r * (gamma + 1));
        if (subset != 0 && (int)(is_migrated[r] != 0) != (subset == 2)) return;
        if (q_indptr) {                                             // ragged rows: the request has its own depth and row offset
            const int64_t r0 = q_indptr[r], n = q_indptr[r + 1] - r0;
            if (n < 1 || n > gamma + 1) {
                if (lane == 0 && t == 0 && kv == 0) {
                    atomicOr(status, STATUS_BAD_TOKEN);
                    atomicCAS(status + 1, 0, r + 1);
                }
                return;
            }
            if (t >= n) return;
            row = r0 + t;
        }
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
        srcv = (kv ? v_new : k_new) + row * sh.Hkv * sh.D;
        dstb = slab + (int64_t)b * sh.block_elems() + (int64_t)kv * sh.Hkv * sh.tile_elems() + (int64_t)slot * sh.D;
    }();
    pdl_wait();
    if (!dstb) return;
    const int vec_per_head = sh.D / 8;                              // 16-byte pieces per head vector
    const int n_vec = sh.Hkv * vec_per_head;
    for (int i = lane; i < n_vec; i += 32) {
        const int h = i / vec_per_head, c = i - h * vec_per_head;
        const int4 v = __ldg(reinterpret_cast<const int4*>(srcv + (int64_t)h * sh.D) + c);
        *(reinterpret_cast<int4*>(dstb + (int64_t)h * sh.tile_elems()) + c) = v;
    }
}

// Suffix commit: one warp per (request, token t <= gamma, K|V); a warp whose token was not
// committed (t > acc_len[r]) leaves at once.  acc_len is read on the device, so the call
// needs no host round trip after the acceptance kernel.
__global__ void __launch_bounds__(256)
commit_suffix_kernel(uint16_t* __restrict__ slab, Shape sh, int32_t batch, int32_t gamma,
                     const int64_t* __restrict__ q_indptr, const int32_t* __restrict__ ctx_len, const int32_t* __restrict__ acc_len,
                     const int64_t* __restrict__ kv_indptr, const int32_t* __restrict__ kv_indices,
                     const int64_t* __restrict__ exp_indptr, const int32_t* __restrict__ exp_indices,
                     int32_t* __restrict__ new_ctx_len, int32_t* __restrict__ status) {
    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t n_rows = (int64_t)batch * (gamma + 1);
    if (warp >= 2 * n_rows) return;
    const int kv = (int)(warp & 1);
    const int64_t row = warp >> 1;
    const int r = (int)(row / (gamma + 1));
    const int t = (int)(row - (int64_t)r * (gamma + 1));
    const int acc = acc_len[r];
    // at most the drafts the request had: gamma, or its own depth when the rows are ragged
    const int depth = q_indptr ? (int)min((int64_t)gamma, q_indptr[r + 1] - q_indptr[r] - 1) : gamma;
    if (acc < 0 || acc > depth) {
        if (lane == 0 && t == 0 && kv == 0) {
            atomicOr(status, STATUS_BAD_TOKEN);
            atomicCAS(status + 1, 0, r + 1);
        }
        return;
    }
    if (new_ctx_len && t == 0 && kv == 0 && lane == 0) new_ctx_len[r] = ctx_len[r] + 1 + acc;
    if (t > acc) return;
    const int64_t pos = (int64_t)ctx_len[r] + t;
    const int64_t j = pos / sh.bs;
    const int slot = (int)(pos - j * sh.bs);
    int32_t from = -1, to = -1;
    if (ctx_len[r] >= 0 && kv_indptr[r] + j < kv_indptr[r + 1] && exp_indptr[r] + j < exp_indptr[r + 1]) {
        from = kv_indices[kv_indptr[r] + j];
        to = exp_indices[exp_indptr[r] + j];
    }
    if ((uint32_t)from >= (uint32_t)sh.num_blocks || (uint32_t)to >= (uint32_t)sh.num_blocks) {
        if (lane == 0) {
            atomicOr(status, STATUS_BAD_BLOCK);
            atomicCAS(status + 1, 0, r + 1);
        }
        return;
    }
    const int64_t in_block = (int64_t)kv * sh.Hkv * sh.tile_elems() + (int64_t)slot * sh.D;
    const uint16_t* srcb = slab + (int64_t)from * sh.block_elems() + in_block;
    uint16_t* dstb = slab + (int64_t)to * sh.block_elems() + in_block;
    const int vec_per_head = sh.D / 8;
    const int n_vec = sh.Hkv * vec_per_head;
    for (int i = lane; i < n_vec; i += 32) {
        const int h = i / vec_per_head, c = i - h * vec_per_head;
        const int4 v = *(reinterpret_cast<const int4*>(srcb + (int64_t)h * sh.tile_elems()) + c);
        *(reinterpret_cast<int4*>(dstb + (int64_t)h * sh.tile_elems()) + c) = v;
    }
}

}  // namespace

cudaError_t gather_init() {
    return cudaFuncSetAttribute(gather_blocks_bulk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kBulkSlots * kBulkBytes);
}

cudaError_t launch_gather(const Shape& s, uint16_t* slab, int64_t n_pairs, const int32_t* src, const int32_t* dst,
                          int32_t* status, int n_sms, uint32_t wait_budget, uint32_t starve_bytes, cudaStream_t stream) {
    if (n_pairs <= 0) return cudaSuccess;
    const int64_t block_bytes = s.block_elems() * 2;
    const int32_t ppb = (int32_t)((block_bytes + kBulkBytes - 1) / kBulkBytes);
    const int64_t n_pieces = n_pairs * ppb;
    // A bounded number of CTAs (4 per SM, each with 48 KiB of loads in flight): the copy shares the SMs with attention.
    const int64_t ctas = (int64_t)(n_sms > 0 ? n_sms : 148) * kBulkCtasPerSm;
    const int grid = (int)(n_pieces < ctas ? n_pieces : ctas);
    gather_blocks_bulk_kernel<<<grid, 32, kBulkSlots * kBulkBytes, stream>>>(slab, n_pairs, src, dst, s.num_blocks, block_bytes, ppb, status,
                                                                          wait_budget ? wait_budget : kBulkSpinLimit, starve_bytes);
    return cudaGetLastError();
}

cudaError_t launch_append(const Shape& s, uint16_t* slab, int32_t batch, int32_t gamma, const int64_t* q_indptr,
                          const int32_t* ctx_len, const int64_t* kv_indptr, const int32_t* kv_indices, const uint16_t* k_new,
                          const uint16_t* v_new, const uint8_t* is_migrated, int32_t subset, int32_t* status,
                          cudaStream_t stream, bool pdl) {
    const int64_t warps = 2LL * batch * (gamma + 1);
    if (warps <= 0) return cudaSuccess;
    const int grid = (int)((warps * 32 + 255) / 256);
    return launch_kernel(append_tokens_kernel, dim3(grid), dim3(256), 0, stream, pdl, slab, s, batch, gamma, q_indptr, ctx_len,
                         kv_indptr, kv_indices, k_new, v_new, is_migrated, subset, status);
}

cudaError_t launch_commit(const Shape& s, uint16_t* slab, int32_t batch, int32_t gamma, const int64_t* q_indptr,
                          const int32_t* ctx_len, const int32_t* acc_len, const int64_t* kv_indptr, const int32_t* kv_indices,
                          const int64_t* exp_indptr, const int32_t* exp_indices, int32_t* new_ctx_len, int32_t* status,
                          cudaStream_t stream) {
    const int64_t warps = 2LL * batch * (gamma + 1);
    if (warps <= 0) return cudaSuccess;
    const int grid = (int)((warps * 32 + 255) / 256);
    commit_suffix_kernel<<<grid, 256, 0, stream>>>(slab, s, batch, gamma, q_indptr, ctx_len, acc_len, kv_indptr, kv_indices, exp_indptr,
                                                   exp_indices, new_ctx_len, status);
    return cudaGetLastError();
}

}  // namespace nsd
