// Internal declarations shared by the library's translation units (not part of the ABI).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "nsd.h"

namespace nsd {

// ---- programmatic dependent launch -------------------------------------------------------------
// A kernel launched with `pdl` may become resident while the kernel before it on the stream is still running (as
// soon as every CTA of that one has let its dependents go, or has exited).  It may read its own inputs and set
// itself up, and must execute pdl_wait() before it touches anything the predecessor writes, or writes anything the
// predecessor still reads; the wait returns when the predecessor grid has completed and its writes are visible.
// Without the attribute both instructions do nothing, so one kernel serves both kinds of launch.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_release_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... P, typename... A>
inline cudaError_t launch_kernel(void (*kernel)(P...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, bool pdl, A... args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<P>(args)...);
}
#endif

// One unit of attention work: a range of KV blocks of one request.  The grid
// runs one CTA per (item, kv head).
struct __align__(16) AttnItem {
    int32_t req;
    int32_t blk_begin;   // first block of the chunk (index into the request's table)
    int32_t blk_end;     // one past the last block
    int32_t part_base;   // first partial slot of the request, -1 when it has a single chunk
    int32_t chunk_idx;
    int32_t nchunks;
    int32_t src_off;     // first entry of the request's source blocks in the gather list, -1 = resident
    int32_t ctx;         // the request's context length when the plan was made (saves the kernels a dependent load)
    int32_t tbl_off;     // kv_indptr[req] when the plan was made (same); -1 = read kv_indptr[req] on the device
    int32_t gamma;       // the request's draft depth: it has gamma + 1 query rows
    int32_t row0;        // its first row in the row tensors (q, o, k_new, v_new): req * (gamma + 1), or the ragged offset
    int32_t pad;
};
static_assert(sizeof(AttnItem) == 48, "AttnItem is read as three 16-byte words");

// Device status word: [0] = error bits, [1] = first offending request (+1; 0 = none).
enum : int32_t { STATUS_BAD_BLOCK = 1, STATUS_BAD_TOKEN = 2, STATUS_TIMEOUT = 4, STATUS_LAYOUT = 8 };

struct Shape {
    int32_t num_slabs, num_blocks, Hq, Hkv, D, bs;
    __host__ __device__ int64_t tile_elems() const { return (int64_t)bs * D; }            // one (block, kv, head)
    __host__ __device__ int64_t block_elems() const { return 2LL * Hkv * bs * D; }        // one (slab, block)
    __host__ __device__ int64_t slab_elems() const { return (int64_t)num_blocks * block_elems(); }
};

struct AttnLaunch {
    Shape shape;
    const uint16_t* pool_slab;   // base of the layer's slab
    // gather-through mode (fuse != 0): items with src_off >= 0 stream their committed KV from the source
    // blocks, take the new tokens from k_new / v_new, and write both to the destination blocks as they go
    int32_t fuse;
    uint16_t* pool_slab_w;
    const int32_t* mig_src;
    const uint16_t* k_new;       // this layer's [rows][Hkv][D]
    const uint16_t* v_new;
    const uint16_t* q;
    uint16_t* o;
    float* lse;
    const int32_t* ctx_len;
    const int64_t* kv_indptr;
    const int32_t* kv_indices;
    const AttnItem* items;
    int32_t n_items;
    int32_t gamma;
    float* part_acc;             // [slot][Hkv][M][D]
    float* part_ml;              // [slot][Hkv][M][2]
    int32_t* counters;           // [max_batch][Hkv], zero between launches
    int32_t* status;
    int32_t m_rows;              // stacked query rows the launch is shaped for: every item has (Hq/Hkv) * (item.gamma+1) <= m_rows
    int32_t m_stride;            // rows per split-KV partial slot (the plan's largest m_rows)
    int32_t tmap_valid;          // tmap describes pool_slab
    int32_t tma_feed;            // mma.sync kernel: fetch K/V tiles with tensor copies where the shape allows
    uint32_t wait_budget;        // polls per bounded barrier wait, 0 = the kernel's default
    int32_t tmap3_valid;         // tmap3 describes pool_slab
    int32_t any_split;           // some request of the plan has more than one chunk (the tcgen05 engine then launches its merge)
    int32_t pdl;                 // host side only: launch as a programmatic dependent of the kernel before it on the stream
    int32_t cta_slots;           // host side only: CTAs the machine holds at once (SMs x resident CTAs); 0 = not known
    CUtensorMap tmap;
    CUtensorMap tmap3;           // tcgen05 engine: 3-D view whose box is a block's whole [16 keys][128 dims] tile
};

// wait_budget: polls per bounded barrier wait (0 = default); starve_bytes: test hook, extra transaction bytes every
// barrier expects and never receives (0 in production).
cudaError_t launch_gather(const Shape& s, uint16_t* slab, int64_t n_pairs, const int32_t* src, const int32_t* dst,
                          int32_t* status, int n_sms, uint32_t wait_budget, uint32_t starve_bytes, cudaStream_t stream);
// q_indptr (nullable, device int64 [batch+1]): ragged rows, request r has q_indptr[r+1] - q_indptr[r] - 1 drafts <= gamma.
cudaError_t launch_append(const Shape& s, uint16_t* slab, int32_t batch, int32_t gamma, const int64_t* q_indptr,
                          const int32_t* ctx_len, const int64_t* kv_indptr, const int32_t* kv_indices, const uint16_t* k_new,
                          const uint16_t* v_new, const uint8_t* is_migrated, int32_t subset, int32_t* status,
                          cudaStream_t stream, bool pdl = false);
cudaError_t launch_commit(const Shape& s, uint16_t* slab, int32_t batch, int32_t gamma, const int64_t* q_indptr,
                          const int32_t* ctx_len, const int32_t* acc_len, const int64_t* kv_indptr, const int32_t* kv_indices,
                          const int64_t* exp_indptr, const int32_t* exp_indices, int32_t* new_ctx_len, int32_t* status,
                          cudaStream_t stream);
cudaError_t launch_attn(const AttnLaunch& a, cudaStream_t stream);
cudaError_t gather_init();        // opt in to the copy ring's dynamic shared memory, once per device
cudaError_t attn_umma_init();     // same for the tcgen05 attention kernels
bool attn_umma_supported(const AttnLaunch& a);
bool attn_umma_preferred(const AttnLaunch& a);   // the shapes where the tcgen05 engine is the faster one
cudaError_t launch_attn_umma(const AttnLaunch& a, cudaStream_t stream, int n_sms);
bool make_kv_tensor_map(CUtensorMap* map, const void* slab, const Shape& s);
bool make_kv_tensor_map3(CUtensorMap* map, const void* slab, const Shape& s);
cudaError_t attn_init();          // opt in to large dynamic shared memory, once per process
// Scratch for sharing one request among several acceptance CTAs (small batches): one row of segment sums and one
// arrival counter (zero between launches) per request.
struct AcceptSplit {
    double* scratch;      // [rows_cap][ceil(vocab_cap / 128)]
    int32_t* counters;    // [rows_cap]
    int32_t rows_cap, vocab_cap, n_sms;
};
cudaError_t launch_accept(const float* p, const float* q, const int32_t* draft_tok, const float* u_acc,
                          const float* u_smp, int32_t batch, int32_t gamma, int32_t vocab, const int64_t* q_indptr,
                          const int32_t* ctx_len, int32_t* acc_len, int32_t* out_tok, int32_t* new_ctx_len, int32_t* status,
                          const AcceptSplit& split, cudaStream_t stream, bool pdl = false);

cudaError_t launch_accept_logits(const void* logits, int32_t logits_bf16, float temperature, const float* q,
                                 const int32_t* draft_tok, const float* u_acc, const float* u_smp, int32_t batch,
                                 int32_t gamma, int32_t vocab, const int32_t* gamma_r, const int32_t* ctx_len,
                                 int32_t* acc_len, int32_t* out_tok, int32_t* new_ctx_len, int32_t* status,
                                 int32_t n_sms, int32_t feed /* 0 = direct loads, 1 = shared-memory ring where aligned */,
                                 int32_t* tickets /* two words, zero between launches */, cudaStream_t stream);

}  // namespace nsd
