// C ABI of the verification-round library: context, host-side validation and
// planning, and the stream choreography of the fused round (Section 4: the
// preparation of state overlaps model execution; Eq. (F.3): a batch runs only
// once its KV state is ready).  See include/nsd.h for the contract.
#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "nsd_internal.h"

using namespace nsd;

constexpr int kAttnClasses = 6;
constexpr int kAttnGroups = 2;

struct nsd_ctx {
    nsd_config cfg;
    Shape shape;
    int device;
    // device workspace carve-up
    char* ws;
    size_t ws_bytes;
    int32_t* d_status;       // [4]
    int32_t* d_counters;     // [max_batch * Hkv]
    AcceptSplit accept_split; // scratch rows and counters for sharing a request among acceptance CTAs
    AttnItem* d_items_all;   // [max_items]
    AttnItem* d_items_split; // [max_items]  resident items then reassigned items
    float* d_part_ml;        // [part_slots * Hkv * Mmax * 2]
    float* d_part_acc;       // [part_slots * Hkv * Mmax * D]
    int64_t max_items, part_slots;
    int32_t m_max;
    // pinned staging for the plan
    AttnItem* h_items;       // [2 * max_items]
    int32_t* h_status;       // [4]
    // current plan
    bool planned;
    int32_t plan_batch, plan_gamma;
    int32_t n_all, n_res, n_mig_items;
    // Items whose stacked query rows need at most four 8-row tiles (bound by HBM whatever their width: one launch shaped
    // for the widest of them) and the wider ones (bound by arithmetic: the tcgen05 engine) form two groups, the wide one
    // first; inside a group the order is longest first.  grp_*[g] .. grp_*[g+1] = the items of group g in the list of all
    // items, in the resident part and in the reassigned part of the split list; rows_*[g] = rows of its widest class.
    int32_t grp_all[kAttnGroups + 1], grp_res[kAttnGroups + 1], grp_mig[kAttnGroups + 1];
    int32_t rows_all[kAttnGroups], rows_res[kAttnGroups], rows_mig[kAttnGroups];
    int64_t plan_rows;         // query rows of the planned batch: batch * (gamma + 1), or the ragged total
    bool plan_ragged;          // the plan was given per-request depths (h_q_indptr)
    int32_t plan_m_stride;     // rows per split-KV partial slot
    int32_t plan_split_slots;  // partial slots the plan uses (0 = no request is split)
    int64_t plan_src_blocks;   // source blocks of the planned batch's reassigned requests
    bool plan_has_mig;         // the plan was given is_migrated (its resident / reassigned item lists are meaningful)
    // streams / events
    cudaStream_t side;
    cudaStream_t copy, down;   // nsd_verify_round_host: uploads in the order they are needed / per-layer read-back of o
    cudaEvent_t ev_start, ev_side_done, ev_plan_free, ev_copy_go, ev_accept_in, ev_tables, ev_down_done;
    std::vector<cudaEvent_t> ev_prep, ev_attn;
    std::vector<cudaEvent_t> ev_in, ev_out;    // nsd_verify_round_host: layer l's inputs have landed / its output is complete
    // tcgen05 attention: one tensor map per layer slab of the pool last seen, and the SM count for the persistent grid
    std::vector<CUtensorMap> tmaps, tmaps3;
    std::vector<const void*> tmap_slab;
    std::vector<char> tmap3_ok;
    int n_sms;
    bool pdl;                  // nsd_verify_round launches its kernels as programmatic dependents of one another
    int round_split;           // first layer of a round with reassigned requests: 0 = by size, 1 = always attend resident and reassigned requests separately, 2 = never
    int logits_feed;           // acceptance from logits: 1 = rows through the shared-memory ring where aligned (default), 0 = direct loads
    int attn_feed_tma;         // mma.sync kernel: K/V tiles by tensor copies where that is the faster feed (default), 0 = cp.async everywhere
    int attn_tcgen05;          // tcgen05 engine: 0 = never, 1 = for the shapes where it is the faster one (default), 2 = wherever it applies
    uint32_t wait_budget;      // polls per bounded wait, 0 = the kernels' default
    uint32_t starve_gather;    // test hook: extra transaction bytes the gather expects and never gets
    int64_t launches;
    char err[256];
};

namespace {

// Row-tile classes of the attention kernel: (warps, 8-row tiles per warp) = 1x1, 1x2, 1x3, 2x2, 2x3, 3x3.
int attn_class_of(int m_rows) {
    const int nt8 = (m_rows + 7) / 8;
    return nt8 <= 3 ? nt8 - 1 : (nt8 == 4 ? 3 : (nt8 <= 6 ? 4 : 5));
}
int attn_class_rows(int cls) {
    static const int rows[kAttnClasses] = {8, 16, 24, 32, 48, 64};
    return rows[cls];
}

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

bool config_ok(const nsd_config* c) {
    if (!c) return false;
    if (c->num_layers < 1 || c->num_slabs < 1 || c->num_slabs > c->num_layers) return false;
    if (c->num_q_heads < 1 || c->num_kv_heads < 1 || c->num_q_heads % c->num_kv_heads) return false;
    if (c->num_blocks < 1 || c->region_b_begin < 0 || c->region_b_begin > c->num_blocks) return false;
    if (c->max_batch < 1 || c->max_gamma < 1 || c->vocab_size < 1 || c->max_table_entries < 1) return false;
    return true;
}
bool config_supported(const nsd_config* c) {
    if (c->head_dim != 64 && c->head_dim != 128) return false;
    if (c->block_size != 16) return false;
    if (c->max_gamma > 31) return false;
    if ((c->num_q_heads / c->num_kv_heads) * (c->max_gamma + 1) > 64) return false;
    return true;
}

struct Layout {
    size_t status, counters, acc_counters, items_all, items_split, acc_scratch, part_ml, part_acc, total;
    int64_t max_items, part_slots;
    int32_t m_max, acc_rows;
};

Layout make_layout(const nsd_config* c) {
    Layout L{};
    L.m_max = (c->num_q_heads / c->num_kv_heads) * (c->max_gamma + 1);
    // An item covers at least kMinChunkBlocks blocks unless it is a request's only or last chunk.
    L.part_slots = std::max<int64_t>(4LL * c->max_batch, 1024);
    L.max_items = (int64_t)c->max_batch + L.part_slots;
    size_t off = 0;
    L.status = off;      off = align_up(off + 4 * sizeof(int32_t), 256);
    L.counters = off;    off = align_up(off + (size_t)c->max_batch * c->num_kv_heads * sizeof(int32_t), 256);
    L.acc_rows = std::min<int32_t>(c->max_batch, 512);                   // requests that may be shared among acceptance CTAs
    L.acc_counters = off; off = align_up(off + (size_t)(L.acc_rows + 2) * sizeof(int32_t), 256);   // + the two request tickets of the logits kernel
    L.items_all = off;   off = align_up(off + (size_t)L.max_items * sizeof(AttnItem), 256);
    L.items_split = off; off = align_up(off + (size_t)L.max_items * sizeof(AttnItem), 256);
    L.acc_scratch = off; off = align_up(off + (size_t)L.acc_rows * ((c->vocab_size + 127) / 128) * sizeof(double), 256);
    L.part_ml = off;     off = align_up(off + (size_t)L.part_slots * c->num_kv_heads * L.m_max * 2 * sizeof(float), 256);
    L.part_acc = off;    off = align_up(off + (size_t)L.part_slots * c->num_kv_heads * L.m_max * c->head_dim * sizeof(float), 256);
    L.total = off;
    return L;
}

nsd_status cuda_fail(nsd_ctx* ctx, cudaError_t e, const char* what) {
    if (ctx) snprintf(ctx->err, sizeof ctx->err, "%.160s: %.80s", what, cudaGetErrorString(e));   // the call's text may be long: keep both parts
    return NSD_ERR_CUDA;
}
#define NSD_CUDA(ctx, call)                                         \
    do {                                                            \
        cudaError_t e__ = (call);                                   \
        if (e__ != cudaSuccess) return cuda_fail(ctx, e__, #call);  \
    } while (0)

uint16_t* slab_ptr(const nsd_ctx* ctx, void* pool, int layer) {
    return static_cast<uint16_t*>(pool) + (int64_t)(layer % ctx->cfg.num_slabs) * ctx->shape.slab_elems();
}

}  // namespace

extern "C" {

const char* nsd_status_string(nsd_status s) {
    switch (s) {
        case NSD_OK: return "ok";
        case NSD_ERR_INVALID_ARG: return "invalid argument";
        case NSD_ERR_OUT_OF_RANGE: return "argument out of configured range";
        case NSD_ERR_CAPACITY: return "capacity exceeded";
        case NSD_ERR_UNSUPPORTED: return "unsupported shape";
        case NSD_ERR_CUDA: return "CUDA runtime error";
        case NSD_ERR_DEVICE_FAULT: return "out-of-range index met on the device";
        case NSD_ERR_NOT_PLANNED: return "no plan for this batch";
        case NSD_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    }
    return "unknown";
}

const char* nsd_last_error(const nsd_ctx* ctx) { return ctx ? ctx->err : ""; }

size_t nsd_workspace_bytes(const nsd_config* cfg) {
    if (!config_ok(cfg) || !config_supported(cfg)) return 0;
    return make_layout(cfg).total;
}

size_t nsd_kv_pool_bytes(const nsd_config* cfg) {
    if (!config_ok(cfg)) return 0;
    return (size_t)cfg->num_slabs * cfg->num_blocks * 2 * cfg->num_kv_heads * cfg->block_size * cfg->head_dim * 2;
}

static nsd_status create_impl(const nsd_config* cfg, void* d_workspace, size_t workspace_bytes, nsd_ctx** out);

nsd_status nsd_create(const nsd_config* cfg, void* d_workspace, size_t workspace_bytes, nsd_ctx** out) {
    try {
        return create_impl(cfg, d_workspace, workspace_bytes, out);
    } catch (...) {                        // host allocation of the event lists failed
        return NSD_ERR_CAPACITY;
    }
}

static nsd_status create_impl(const nsd_config* cfg, void* d_workspace, size_t workspace_bytes, nsd_ctx** out) {
    if (!out) return NSD_ERR_INVALID_ARG;
    *out = nullptr;
    if (!config_ok(cfg) || !d_workspace) return NSD_ERR_INVALID_ARG;
    if (!config_supported(cfg)) return NSD_ERR_UNSUPPORTED;
    if (reinterpret_cast<uintptr_t>(d_workspace) % 256) return NSD_ERR_INVALID_ARG;
    const Layout L = make_layout(cfg);
    if (workspace_bytes < L.total) return NSD_ERR_CAPACITY;

    nsd_ctx* ctx = new (std::nothrow) nsd_ctx();
    if (!ctx) return NSD_ERR_CAPACITY;
    ctx->cfg = *cfg;
    ctx->shape = Shape{cfg->num_slabs, cfg->num_blocks, cfg->num_q_heads, cfg->num_kv_heads, cfg->head_dim, cfg->block_size};
    ctx->ws = static_cast<char*>(d_workspace);
    ctx->ws_bytes = L.total;
    ctx->d_status = reinterpret_cast<int32_t*>(ctx->ws + L.status);
    ctx->d_counters = reinterpret_cast<int32_t*>(ctx->ws + L.counters);
    ctx->d_items_all = reinterpret_cast<AttnItem*>(ctx->ws + L.items_all);
    ctx->d_items_split = reinterpret_cast<AttnItem*>(ctx->ws + L.items_split);
    ctx->d_part_ml = reinterpret_cast<float*>(ctx->ws + L.part_ml);
    ctx->accept_split = AcceptSplit{reinterpret_cast<double*>(ctx->ws + L.acc_scratch), reinterpret_cast<int32_t*>(ctx->ws + L.acc_counters),
                                    L.acc_rows, cfg->vocab_size, 0};
    ctx->d_part_acc = reinterpret_cast<float*>(ctx->ws + L.part_acc);
    ctx->max_items = L.max_items;
    ctx->part_slots = L.part_slots;
    ctx->m_max = L.m_max;
    ctx->planned = false;
    ctx->launches = 0;
    ctx->err[0] = 0;
    ctx->h_items = nullptr;
    ctx->h_status = nullptr;
    ctx->side = nullptr;
    ctx->copy = nullptr;
    ctx->ev_start = ctx->ev_side_done = ctx->ev_plan_free = ctx->ev_copy_go = ctx->ev_accept_in = ctx->ev_tables = ctx->ev_down_done = nullptr;
    ctx->down = nullptr;

    auto fail = [&](cudaError_t e, const char* what) {
        nsd_status s = cuda_fail(ctx, e, what);
        fprintf(stderr, "nsd_create: %s\n", ctx->err);
        nsd_destroy(ctx);
        return s;
    };
    cudaError_t e;
    if ((e = cudaGetDevice(&ctx->device)) != cudaSuccess) return fail(e, "cudaGetDevice");
    // zero the bookkeeping part of the workspace (status, counters, work lists); partials need no init
    if ((e = cudaMemset(ctx->ws, 0, L.part_ml)) != cudaSuccess) return fail(e, "cudaMemset(workspace)");
    if ((e = cudaDeviceSynchronize()) != cudaSuccess) return fail(e, "cudaDeviceSynchronize");
    if ((e = cudaMallocHost(&ctx->h_items, 2 * (size_t)L.max_items * sizeof(AttnItem))) != cudaSuccess) return fail(e, "cudaMallocHost(items)");
    if ((e = cudaMallocHost(&ctx->h_status, 4 * sizeof(int32_t))) != cudaSuccess) return fail(e, "cudaMallocHost(status)");
    if ((e = cudaStreamCreateWithFlags(&ctx->side, cudaStreamNonBlocking)) != cudaSuccess) return fail(e, "cudaStreamCreate");
    if ((e = cudaStreamCreateWithFlags(&ctx->copy, cudaStreamNonBlocking)) != cudaSuccess) return fail(e, "cudaStreamCreate");
    if ((e = cudaStreamCreateWithFlags(&ctx->down, cudaStreamNonBlocking)) != cudaSuccess) return fail(e, "cudaStreamCreate");
    if ((e = cudaEventCreateWithFlags(&ctx->ev_tables, cudaEventDisableTiming)) != cudaSuccess) return fail(e, "cudaEventCreate");
    if ((e = cudaEventCreateWithFlags(&ctx->ev_down_done, cudaEventDisableTiming)) != cudaSuccess) return fail(e, "cudaEventCreate");
    if ((e = cudaEventCreateWithFlags(&ctx->ev_copy_go, cudaEventDisableTiming)) != cudaSuccess) return fail(e, "cudaEventCreate");
    if ((e = cudaEventCreateWithFlags(&ctx->ev_accept_in, cudaEventDisableTiming)) != cudaSuccess) return fail(e, "cudaEventCreate");
    if ((e = cudaEventCreateWithFlags(&ctx->ev_start, cudaEventDisableTiming)) != cudaSuccess) return fail(e, "cudaEventCreate");
    if ((e = cudaEventCreateWithFlags(&ctx->ev_side_done, cudaEventDisableTiming)) != cudaSuccess) return fail(e, "cudaEventCreate");
    if ((e = cudaEventCreateWithFlags(&ctx->ev_plan_free, cudaEventDisableTiming)) != cudaSuccess) return fail(e, "cudaEventCreate");
    ctx->ev_prep.assign(cfg->num_layers, nullptr);
    ctx->ev_attn.assign(cfg->num_layers, nullptr);
    ctx->ev_in.assign(cfg->num_layers, nullptr);
    ctx->ev_out.assign(cfg->num_layers, nullptr);
    for (int l = 0; l < cfg->num_layers; ++l) {
        if ((e = cudaEventCreateWithFlags(&ctx->ev_prep[l], cudaEventDisableTiming)) != cudaSuccess) return fail(e, "cudaEventCreate");
        if ((e = cudaEventCreateWithFlags(&ctx->ev_attn[l], cudaEventDisableTiming)) != cudaSuccess) return fail(e, "cudaEventCreate");
        if ((e = cudaEventCreateWithFlags(&ctx->ev_in[l], cudaEventDisableTiming)) != cudaSuccess) return fail(e, "cudaEventCreate");
        if ((e = cudaEventCreateWithFlags(&ctx->ev_out[l], cudaEventDisableTiming)) != cudaSuccess) return fail(e, "cudaEventCreate");
    }
    if ((e = attn_init()) != cudaSuccess) return fail(e, "cudaFuncSetAttribute(attention)");
    if ((e = gather_init()) != cudaSuccess) return fail(e, "cudaFuncSetAttribute(gather)");
    if ((e = attn_umma_init()) != cudaSuccess) return fail(e, "cudaFuncSetAttribute(tcgen05 attention)");
    ctx->tmaps.resize(cfg->num_slabs);
    ctx->tmaps3.resize(cfg->num_slabs);
    ctx->tmap3_ok.assign(cfg->num_slabs, 0);
    ctx->tmap_slab.assign(cfg->num_slabs, nullptr);
    if ((e = cudaDeviceGetAttribute(&ctx->n_sms, cudaDevAttrMultiProcessorCount, ctx->device)) != cudaSuccess) return fail(e, "cudaDeviceGetAttribute");
    ctx->accept_split.n_sms = ctx->n_sms;
    // Kernel selection (cfg->flags): the defaults are the faster kernel for each shape.
    ctx->attn_feed_tma = !(cfg->flags & NSD_FLAG_ATTN_CP_ASYNC);
    ctx->attn_tcgen05 = (cfg->flags & NSD_FLAG_ATTN_NO_TCGEN05) ? 0 : ((cfg->flags & NSD_FLAG_ATTN_TCGEN05) ? 2 : 1);
    ctx->round_split = (cfg->flags & NSD_FLAG_ROUND_SPLIT_ALWAYS) ? 1 : ((cfg->flags & NSD_FLAG_ROUND_SPLIT_NEVER) ? 2 : 0);
    ctx->logits_feed = (cfg->flags & NSD_FLAG_LOGITS_DIRECT) ? 0 : 1;
    ctx->pdl = !(cfg->flags & NSD_FLAG_NO_DEPENDENT_LAUNCH);
    ctx->wait_budget = cfg->wait_budget > 0 ? (uint32_t)cfg->wait_budget : 0u;
    ctx->starve_gather = (cfg->flags & NSD_FLAG_TEST_STARVE_GATHER) ? 16u : 0u;
    *out = ctx;
    return NSD_OK;
}

nsd_status nsd_destroy(nsd_ctx* ctx) {
    if (!ctx) return NSD_OK;
    if (ctx->side) { cudaStreamSynchronize(ctx->side); cudaStreamDestroy(ctx->side); }
    if (ctx->copy) { cudaStreamSynchronize(ctx->copy); cudaStreamDestroy(ctx->copy); }
    if (ctx->down) { cudaStreamSynchronize(ctx->down); cudaStreamDestroy(ctx->down); }
    if (ctx->ev_tables) cudaEventDestroy(ctx->ev_tables);
    if (ctx->ev_down_done) cudaEventDestroy(ctx->ev_down_done);
    for (auto ev : ctx->ev_in) if (ev) cudaEventDestroy(ev);
    for (auto ev : ctx->ev_out) if (ev) cudaEventDestroy(ev);
    if (ctx->ev_copy_go) cudaEventDestroy(ctx->ev_copy_go);
    if (ctx->ev_accept_in) cudaEventDestroy(ctx->ev_accept_in);
    for (auto ev : ctx->ev_prep) if (ev) cudaEventDestroy(ev);
    for (auto ev : ctx->ev_attn) if (ev) cudaEventDestroy(ev);
    if (ctx->ev_start) cudaEventDestroy(ctx->ev_start);
    if (ctx->ev_side_done) cudaEventDestroy(ctx->ev_side_done);
    if (ctx->ev_plan_free) cudaEventDestroy(ctx->ev_plan_free);
    if (ctx->h_items) cudaFreeHost(ctx->h_items);
    if (ctx->h_status) cudaFreeHost(ctx->h_status);
    delete ctx;
    return NSD_OK;
}

static nsd_status verify_plan_impl(nsd_ctx* ctx, int32_t batch, int32_t gamma, const int32_t* h_ctx_len,
                                   const int64_t* h_kv_indptr, const uint8_t* h_is_migrated, const int64_t* h_q_indptr,
                                   int32_t chunk_blocks, void* stream);

nsd_status nsd_verify_plan(nsd_ctx* ctx, int32_t batch, int32_t gamma, const int32_t* h_ctx_len,
                           const int64_t* h_kv_indptr, const uint8_t* h_is_migrated, const int64_t* h_q_indptr,
                           int32_t chunk_blocks, void* stream) {
    try {
        return verify_plan_impl(ctx, batch, gamma, h_ctx_len, h_kv_indptr, h_is_migrated, h_q_indptr, chunk_blocks, stream);
    } catch (...) {                        // the host work list could not be allocated: nothing crosses the C boundary
        return NSD_ERR_CAPACITY;
    }
}

static nsd_status verify_plan_impl(nsd_ctx* ctx, int32_t batch, int32_t gamma, const int32_t* h_ctx_len,
                                   const int64_t* h_kv_indptr, const uint8_t* h_is_migrated, const int64_t* h_q_indptr,
                                   int32_t chunk_blocks, void* stream) {
    if (!ctx) return NSD_ERR_INVALID_ARG;
    if (batch < 0 || batch > ctx->cfg.max_batch || gamma < 1 || gamma > ctx->cfg.max_gamma) return NSD_ERR_OUT_OF_RANGE;
    if (chunk_blocks < 0 || (chunk_blocks & 1) || chunk_blocks > 256) return NSD_ERR_INVALID_ARG;
    if (batch > 0 && (!h_ctx_len || !h_kv_indptr)) return NSD_ERR_INVALID_ARG;
    const int bs = ctx->cfg.block_size;
    const int Hkv = ctx->cfg.num_kv_heads;
    // ---- validate lengths and tables
    std::vector<int32_t> nblk(batch), depth(batch, gamma);
    std::vector<int64_t> row0(batch + 1, 0);
    int64_t total_blocks = 0;
    if (batch > 0 && h_q_indptr && h_q_indptr[0] != 0) return NSD_ERR_INVALID_ARG;
    for (int r = 0; r < batch; ++r) {
        if (h_q_indptr) {                                                   // per-request draft depth, rows ragged
            const int64_t n = h_q_indptr[r + 1] - h_q_indptr[r];
            if (n < 1 || n > gamma + 1) return NSD_ERR_OUT_OF_RANGE;
            depth[r] = (int32_t)n - 1;
        }
        row0[r + 1] = row0[r] + depth[r] + 1;
        if (h_ctx_len[r] < 0 || h_kv_indptr[r] < 0 || h_kv_indptr[r + 1] < h_kv_indptr[r]) return NSD_ERR_INVALID_ARG;
        const int64_t need = ((int64_t)h_ctx_len[r] + depth[r] + 1 + bs - 1) / bs;
        if (h_kv_indptr[r + 1] - h_kv_indptr[r] < need) return NSD_ERR_INVALID_ARG;
        if (need > INT32_MAX / 2) return NSD_ERR_OUT_OF_RANGE;
        nblk[r] = (int32_t)need;
        total_blocks += need;
    }
    if (batch > 0 && h_kv_indptr[batch] > ctx->cfg.max_table_entries) return NSD_ERR_CAPACITY;
    if (batch > 0 && h_kv_indptr[batch] > INT32_MAX) return NSD_ERR_CAPACITY;      // items carry table offsets as int32
    if (row0[batch] > INT32_MAX / 2) return NSD_ERR_CAPACITY;                       // ... and row offsets

    // ---- chunk length: split only as far as it takes to give every resident CTA slot of the machine one item.
    //      Measured: a split costs a partial store, a counter and a merge (several microseconds at the end of a
    //      CTA), so one wave of longer chunks beats three waves of short ones at every batch size (batch 64:
    //      101 us against 131 us per layer; batch 512: 408 against 417).
    int cb = chunk_blocks;
    if (cb == 0) {
        const int64_t target_items = (int64_t)ctx->n_sms * 6;          // SMs x resident CTAs
        int64_t want = (total_blocks * Hkv + target_items - 1) / target_items;
        want = std::min<int64_t>(std::max<int64_t>(want, 16), 256);
        cb = (int)((want + 1) & ~1LL);
        // Cutting each request into equal chunks of at most cb blocks rounds the item count up; where one wave is
        // within reach (batch x kv heads fits the slots) lengthen the chunks until the items really fit it: a second
        // wave of a few left-over CTAs costs far more than slightly longer chunks (batch 64: 1.13 waves before).
        if ((int64_t)batch * Hkv <= target_items) {
            auto n_items = [&](int c) {
                int64_t n = 0;
                for (int r = 0; r < batch; ++r) n += (nblk[r] + c - 1) / c;
                return n;
            };
            while (cb < 256 && n_items(cb) * Hkv > target_items) cb += 2;
        }
    }
    auto count_slots = [&](int c) {
        int64_t slots = 0;
        for (int r = 0; r < batch; ++r) {
            const int n = (nblk[r] + c - 1) / c;
            if (n > 1) slots += n;
        }
        return slots;
    };
    while (count_slots(cb) > ctx->part_slots) {
        if (chunk_blocks != 0 || cb >= 256) return NSD_ERR_CAPACITY;
        cb = std::min(256, cb * 2);
    }
    // ---- items
    const int G = ctx->cfg.num_q_heads / ctx->cfg.num_kv_heads;
    struct Tmp { AttnItem it; int mig; int cls; };
    std::vector<Tmp> items;
    int32_t slot = 0;
    int64_t src_next = 0;                                                // running offset into the gather's pair list
    for (int r = 0; r < batch; ++r) {
        const bool mig = h_is_migrated && h_is_migrated[r] != 0;
        const int64_t src_off = mig ? src_next : -1;
        if (mig) src_next += ((int64_t)h_ctx_len[r] + bs - 1) / bs;
        if (src_next > INT32_MAX) return NSD_ERR_CAPACITY;
        const int n = (nblk[r] + cb - 1) / cb;
        int per = (nblk[r] + n - 1) / n;
        per = (per + 1) & ~1;                                            // even: tiles are two blocks
        const int n_eff = (nblk[r] + per - 1) / per;
        const int base = n_eff > 1 ? slot : -1;
        for (int c = 0; c < n_eff; ++c) {
            AttnItem it{};
            it.req = r;
            it.blk_begin = c * per;
            it.blk_end = std::min(nblk[r], (c + 1) * per);
            it.part_base = base;
            it.chunk_idx = c;
            it.nchunks = n_eff;
            it.src_off = (int32_t)src_off;
            it.ctx = h_ctx_len[r];
            it.tbl_off = (int32_t)h_kv_indptr[r];
            it.gamma = depth[r];
            it.row0 = (int32_t)row0[r];
            items.push_back({it, h_is_migrated ? (h_is_migrated[r] != 0) : 0, attn_class_of(G * (depth[r] + 1))});
        }
        if (n_eff > 1) slot += n_eff;
    }
    if ((int64_t)items.size() > ctx->max_items || slot > ctx->part_slots) return NSD_ERR_CAPACITY;
    auto longer = [](const Tmp& a, const Tmp& b) {
        if ((a.cls >= 4) != (b.cls >= 4)) return a.cls >= 4;                  // the wide group first
        const int la = a.it.blk_end - a.it.blk_begin, lb = b.it.blk_end - b.it.blk_begin;
        if (la != lb) return la > lb;
        if (a.it.req != b.it.req) return a.it.req < b.it.req;
        return a.it.chunk_idx < b.it.chunk_idx;
    };
    std::sort(items.begin(), items.end(), longer);

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // the pinned staging may still be the source of the previous plan's copy
    NSD_CUDA(ctx, cudaEventSynchronize(ctx->ev_plan_free));
    const int n_all = (int)items.size();
    int n_res = 0;
    for (int i = 0; i < n_all; ++i) ctx->h_items[i] = items[i].it;
    AttnItem* split = ctx->h_items + ctx->max_items;
    for (int i = 0; i < n_all; ++i) if (!items[i].mig) split[n_res++] = items[i].it;
    int k = n_res;
    for (int i = 0; i < n_all; ++i) if (items[i].mig) split[k++] = items[i].it;
    if (n_all > 0) {
        NSD_CUDA(ctx, cudaMemcpyAsync(ctx->d_items_all, ctx->h_items, (size_t)n_all * sizeof(AttnItem), cudaMemcpyHostToDevice, st));
        NSD_CUDA(ctx, cudaMemcpyAsync(ctx->d_items_split, split, (size_t)n_all * sizeof(AttnItem), cudaMemcpyHostToDevice, st));
    }
    NSD_CUDA(ctx, cudaEventRecord(ctx->ev_plan_free, st));
    {
        // group boundaries of the three lists and the widest class of each group
        auto bounds = [&](int32_t* off, int32_t* rows, int mig_filter) {
            int32_t count[kAttnGroups] = {0, 0};
            int widest[kAttnGroups] = {-1, -1};
            for (const Tmp& t : items)
                if (mig_filter < 0 || t.mig == mig_filter) {
                    const int g = t.cls >= 4 ? 0 : 1;                       // list position: wide group first
                    count[g]++;
                    widest[g] = std::max(widest[g], t.cls);
                }
            off[0] = 0;
            off[1] = count[0];
            off[2] = count[0] + count[1];
            for (int g = 0; g < kAttnGroups; ++g) rows[g] = widest[g] >= 0 ? attn_class_rows(widest[g]) : 0;
        };
        bounds(ctx->grp_all, ctx->rows_all, -1);
        bounds(ctx->grp_res, ctx->rows_res, 0);
        bounds(ctx->grp_mig, ctx->rows_mig, 1);
    }
    ctx->plan_rows = row0[batch];
    ctx->plan_ragged = h_q_indptr != nullptr;
    ctx->plan_m_stride = G * (gamma + 1);
    ctx->planned = true;
    ctx->plan_batch = batch;
    ctx->plan_gamma = gamma;
    ctx->n_all = n_all;
    ctx->n_res = n_res;
    ctx->n_mig_items = n_all - n_res;
    ctx->plan_src_blocks = src_next;
    ctx->plan_split_slots = slot;
    ctx->plan_has_mig = h_is_migrated != nullptr;
    return NSD_OK;
}

nsd_status nsd_kv_prepare(nsd_ctx* ctx, void* kv_pool, int64_t n_mig_blocks,
                          const int32_t* mig_src, const int32_t* mig_dst, int32_t batch, int32_t gamma,
                          const int32_t* ctx_len, const int64_t* kv_indptr, const int32_t* kv_indices,
                          const void* k_new, const void* v_new, const uint8_t* is_migrated,
                          int32_t append_subset, int32_t layer_begin, int32_t layer_count, const int64_t* q_indptr,
                          int64_t total_rows, void* stream) {
    if (!ctx || !kv_pool) return NSD_ERR_INVALID_ARG;
    if (n_mig_blocks < 0 || layer_count < 0) return NSD_ERR_INVALID_ARG;
    if (batch < 0 || batch > ctx->cfg.max_batch) return NSD_ERR_OUT_OF_RANGE;
    if (layer_begin < 0 || layer_begin + (int64_t)layer_count > ctx->cfg.num_layers) return NSD_ERR_OUT_OF_RANGE;
    const bool do_append = (k_new != nullptr) || (v_new != nullptr);
    if (do_append) {
        if (!k_new || !v_new || !ctx_len || !kv_indptr || !kv_indices) return NSD_ERR_INVALID_ARG;
        if (gamma < 1 || gamma > ctx->cfg.max_gamma) return NSD_ERR_OUT_OF_RANGE;
        if (append_subset < 0 || append_subset > 2 || (append_subset != 0 && !is_migrated)) return NSD_ERR_INVALID_ARG;
    }
    if (n_mig_blocks > 0 && (!mig_src || !mig_dst)) return NSD_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int64_t n_pairs = n_mig_blocks;
    if (q_indptr && (total_rows < batch || total_rows > (int64_t)batch * (gamma + 1))) return NSD_ERR_INVALID_ARG;
    const int64_t layer_rows = (q_indptr ? total_rows : (int64_t)batch * (gamma + 1)) * ctx->cfg.num_kv_heads * ctx->cfg.head_dim;
    for (int l = layer_begin; l < layer_begin + layer_count; ++l) {
        uint16_t* slab = slab_ptr(ctx, kv_pool, l);
        if (n_pairs > 0) {
            NSD_CUDA(ctx, launch_gather(ctx->shape, slab, n_pairs, mig_src, mig_dst, ctx->d_status, ctx->n_sms, ctx->wait_budget, ctx->starve_gather, st));
            ctx->launches++;
        }
        if (do_append && batch > 0) {
            NSD_CUDA(ctx, launch_append(ctx->shape, slab, batch, gamma, q_indptr, ctx_len, kv_indptr, kv_indices,
                                        static_cast<const uint16_t*>(k_new) + (int64_t)l * layer_rows,
                                        static_cast<const uint16_t*>(v_new) + (int64_t)l * layer_rows, is_migrated,
                                        append_subset, ctx->d_status, st));
            ctx->launches++;
        }
    }
    return NSD_OK;
}

nsd_status nsd_kv_commit(nsd_ctx* ctx, void* kv_pool, int32_t batch, int32_t gamma, const int32_t* ctx_len,
                         const int32_t* acc_len, const int64_t* kv_indptr, const int32_t* kv_indices,
                         const int64_t* exp_indptr, const int32_t* exp_indices, int32_t* new_ctx_len,
                         int32_t layer_begin, int32_t layer_count, const int64_t* q_indptr, void* stream) {
    if (!ctx) return NSD_ERR_INVALID_ARG;
    if (batch < 0 || batch > ctx->cfg.max_batch || gamma < 1 || gamma > ctx->cfg.max_gamma) return NSD_ERR_OUT_OF_RANGE;
    if (layer_count < 0) return NSD_ERR_INVALID_ARG;
    if (layer_begin < 0 || layer_begin + (int64_t)layer_count > ctx->cfg.num_layers) return NSD_ERR_OUT_OF_RANGE;
    if (batch == 0 || layer_count == 0) return NSD_OK;
    if (!kv_pool || !ctx_len || !acc_len || !kv_indptr || !kv_indices || !exp_indptr || !exp_indices) return NSD_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    for (int l = layer_begin; l < layer_begin + layer_count; ++l) {
        NSD_CUDA(ctx, launch_commit(ctx->shape, slab_ptr(ctx, kv_pool, l), batch, gamma, q_indptr, ctx_len, acc_len, kv_indptr,
                                    kv_indices, exp_indptr, exp_indices, l == layer_begin ? new_ctx_len : nullptr,
                                    ctx->d_status, st));
        ctx->launches++;
    }
    return NSD_OK;
}

namespace {
struct FuseArgs {
    const int32_t* mig_src;
    const uint16_t* k_new;     // this layer's rows
    const uint16_t* v_new;
};

nsd_status attn_enqueue(nsd_ctx* ctx, const void* kv_pool, const void* q, void* o, float* lse, int32_t gamma,
                        const int32_t* ctx_len, const int64_t* kv_indptr, const int32_t* kv_indices, int32_t layer,
                        int32_t subset, cudaStream_t st, const FuseArgs* fuse = nullptr, bool pdl = false) {
    // pdl: the first launch follows a kernel of the same call on the stream and may be launched as its programmatic dependent
    AttnLaunch a{};
    if (fuse) {
        a.fuse = 1;
        a.pool_slab_w = slab_ptr(ctx, const_cast<void*>(kv_pool), layer);
        a.mig_src = fuse->mig_src;
        a.k_new = fuse->k_new;
        a.v_new = fuse->v_new;
    }
    a.shape = ctx->shape;
    a.pool_slab = slab_ptr(ctx, const_cast<void*>(kv_pool), layer);
    a.q = static_cast<const uint16_t*>(q);
    a.o = static_cast<uint16_t*>(o);
    a.lse = lse;
    a.ctx_len = ctx_len;
    a.kv_indptr = kv_indptr;
    a.kv_indices = kv_indices;
    a.gamma = gamma;
    a.part_acc = ctx->d_part_acc;
    a.part_ml = ctx->d_part_ml;
    a.counters = ctx->d_counters;
    a.status = ctx->d_status;
    a.m_stride = ctx->plan_m_stride;
    a.wait_budget = ctx->wait_budget;
    a.any_split = ctx->plan_split_slots > 0;
    a.cta_slots = ctx->n_sms * 6;
    const AttnItem* base = subset == 0 ? ctx->d_items_all : (subset == 1 ? ctx->d_items_split : ctx->d_items_split + ctx->n_res);
    const int32_t* grp = subset == 0 ? ctx->grp_all : (subset == 1 ? ctx->grp_res : ctx->grp_mig);
    const int32_t* grp_rows = subset == 0 ? ctx->rows_all : (subset == 1 ? ctx->rows_res : ctx->rows_mig);
    if (grp[kAttnGroups] == 0) return NSD_OK;
    if ((ctx->attn_feed_tma || ctx->attn_tcgen05) && ctx->cfg.head_dim == 128) {
        const int slab = layer % ctx->cfg.num_slabs;
        if (ctx->tmap_slab[slab] != a.pool_slab) {
            ctx->tmap_slab[slab] = make_kv_tensor_map(&ctx->tmaps[slab], a.pool_slab, ctx->shape) ? a.pool_slab : nullptr;
            ctx->tmap3_ok[slab] = ctx->attn_tcgen05 && ctx->tmap_slab[slab] && make_kv_tensor_map3(&ctx->tmaps3[slab], a.pool_slab, ctx->shape);
        }
        if (ctx->tmap_slab[slab] == a.pool_slab) {
            a.tmap = ctx->tmaps[slab];
            a.tmap_valid = 1;
            if (ctx->tmap3_ok[slab]) {
                a.tmap3 = ctx->tmaps3[slab];
                a.tmap3_valid = 1;
            }
        }
        a.tma_feed = ctx->attn_feed_tma;
    }
    // one launch per group present (a batch of one draft depth has one), each shaped for its widest item
    for (int pos = 0; pos < kAttnGroups; ++pos) {
        const int n = grp[pos + 1] - grp[pos];
        if (n == 0) continue;
        a.items = base + grp[pos];
        a.n_items = n;
        a.m_rows = std::min(grp_rows[pos], ctx->plan_m_stride);
        if (a.tmap_valid && ctx->attn_tcgen05 && attn_umma_supported(a) && (ctx->attn_tcgen05 == 2 || attn_umma_preferred(a))) {
            NSD_CUDA(ctx, launch_attn_umma(a, st, ctx->n_sms));
            ctx->launches += a.any_split ? 2 : 1;                            // the engine's merge kernel follows when a request is split
            pdl = ctx->pdl;                                                  // what comes next follows a kernel of this call
            continue;
        }
        a.pdl = pdl;
        pdl = ctx->pdl;
        NSD_CUDA(ctx, launch_attn(a, st));
        ctx->launches++;
    }
    return NSD_OK;
}
}  // namespace

nsd_status nsd_verify_attn(nsd_ctx* ctx, const void* kv_pool, const void* q, void* o, float* lse,
                           int32_t batch, int32_t gamma, const int32_t* ctx_len, const int64_t* kv_indptr,
                           const int32_t* kv_indices, int32_t layer, int32_t subset, void* stream) {
    if (!ctx) return NSD_ERR_INVALID_ARG;
    if (batch < 0 || batch > ctx->cfg.max_batch || gamma < 1 || gamma > ctx->cfg.max_gamma) return NSD_ERR_OUT_OF_RANGE;
    if (layer < 0 || layer >= ctx->cfg.num_layers) return NSD_ERR_OUT_OF_RANGE;
    if (subset < 0 || subset > 2) return NSD_ERR_INVALID_ARG;
    if (!ctx->planned || ctx->plan_batch != batch || ctx->plan_gamma != gamma) return NSD_ERR_NOT_PLANNED;
    if (batch == 0) return NSD_OK;
    if (!kv_pool || !q || !o || !ctx_len || !kv_indptr || !kv_indices) return NSD_ERR_INVALID_ARG;
    return attn_enqueue(ctx, kv_pool, q, o, lse, gamma, ctx_len, kv_indptr, kv_indices, layer, subset,
                        static_cast<cudaStream_t>(stream));
}

nsd_status nsd_spec_accept(nsd_ctx* ctx, const float* p, const float* q, const int32_t* draft_tok,
                           const float* u_acc, const float* u_smp, int32_t batch, int32_t gamma, int32_t vocab,
                           const int32_t* ctx_len, int32_t* acc_len, int32_t* out_tok, int32_t* new_ctx_len,
                           const int64_t* q_indptr, void* stream) {
    if (!ctx) return NSD_ERR_INVALID_ARG;
    if (batch < 0 || batch > ctx->cfg.max_batch || gamma < 1 || gamma > ctx->cfg.max_gamma || vocab < 1) return NSD_ERR_OUT_OF_RANGE;
    if (batch == 0) return NSD_OK;
    if (!p || !q || !draft_tok || !u_acc || !u_smp || !acc_len || !out_tok) return NSD_ERR_INVALID_ARG;
    if ((new_ctx_len != nullptr) && !ctx_len) return NSD_ERR_INVALID_ARG;
    NSD_CUDA(ctx, launch_accept(p, q, draft_tok, u_acc, u_smp, batch, gamma, vocab, q_indptr, ctx_len, acc_len, out_tok,
                                new_ctx_len, ctx->d_status, ctx->accept_split, static_cast<cudaStream_t>(stream)));
    ctx->launches++;
    return NSD_OK;
}

nsd_status nsd_spec_accept_logits(nsd_ctx* ctx, const void* logits, int32_t logits_dtype, float temperature,
                                  const float* q, const int32_t* draft_tok, const float* u_acc, const float* u_smp,
                                  int32_t batch, int32_t gamma, int32_t vocab, const int32_t* gamma_r,
                                  const int32_t* ctx_len, int32_t* acc_len, int32_t* out_tok, int32_t* new_ctx_len,
                                  void* stream) {
    if (!ctx) return NSD_ERR_INVALID_ARG;
    if (batch < 0 || batch > ctx->cfg.max_batch || gamma < 1 || gamma > ctx->cfg.max_gamma || vocab < 1) return NSD_ERR_OUT_OF_RANGE;
    if (logits_dtype != 0 && logits_dtype != 1) return NSD_ERR_UNSUPPORTED;
    if (!(temperature >= 0.f)) return NSD_ERR_INVALID_ARG;                       // negative or NaN
    if (batch == 0) return NSD_OK;
    if (!logits || !draft_tok || !acc_len || !out_tok) return NSD_ERR_INVALID_ARG;
    if (temperature > 0.f && (!q || !u_acc || !u_smp)) return NSD_ERR_INVALID_ARG;
    if ((new_ctx_len != nullptr) && !ctx_len) return NSD_ERR_INVALID_ARG;
    NSD_CUDA(ctx, launch_accept_logits(logits, logits_dtype, temperature, q, draft_tok, u_acc, u_smp, batch, gamma, vocab,
                                       gamma_r, ctx_len, acc_len, out_tok, new_ctx_len, ctx->d_status, ctx->n_sms,
                                       ctx->logits_feed, ctx->accept_split.counters + ctx->accept_split.rows_cap,
                                       static_cast<cudaStream_t>(stream)));
    ctx->launches++;
    return NSD_OK;
}

namespace {
// What the host-buffer variant threads through the round: every layer waits for its own inputs (uploaded on the
// copy stream in the order of use), its output is read back on a third stream as soon as it is complete, and the
// acceptance waits for its inputs, which follow the layers' on the copy stream.
struct BeforeAccept {
    void* h_o;                 // host destination of the attention output
    size_t o_layer_bytes;
    cudaEvent_t inputs_ready;  // the acceptance inputs have landed
};
nsd_status round_impl(nsd_ctx* ctx, const nsd_round_args* a, void* stream, const BeforeAccept* hook);
}  // namespace

nsd_status nsd_verify_round(nsd_ctx* ctx, const nsd_round_args* a, void* stream) {
    return round_impl(ctx, a, stream, nullptr);
}

namespace {
nsd_status round_impl(nsd_ctx* ctx, const nsd_round_args* a, void* stream, const BeforeAccept* hook) {
    if (!ctx || !a) return NSD_ERR_INVALID_ARG;
    const int32_t batch = a->batch, gamma = a->gamma;
    if (batch < 0 || batch > ctx->cfg.max_batch || gamma < 1 || gamma > ctx->cfg.max_gamma) return NSD_ERR_OUT_OF_RANGE;
    if (!ctx->planned || ctx->plan_batch != batch || ctx->plan_gamma != gamma) return NSD_ERR_NOT_PLANNED;
    if (batch == 0) return NSD_OK;
    if (!a->kv_pool || !a->ctx_len || !a->kv_indptr || !a->kv_indices || !a->k_new || !a->v_new || !a->q || !a->o ||
        !a->p || !a->q_draft || !a->draft_tok || !a->u_acc || !a->u_smp || !a->acc_len || !a->out_tok)
        return NSD_ERR_INVALID_ARG;
    if (a->n_mig_blocks < 0) return NSD_ERR_INVALID_ARG;
    if (a->n_mig_blocks > 0 && (!a->mig_src || !a->mig_dst || !a->is_migrated)) return NSD_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int L = ctx->cfg.num_layers, S = ctx->cfg.num_slabs;
    const int Hq = ctx->cfg.num_q_heads, Hkv = ctx->cfg.num_kv_heads, D = ctx->cfg.head_dim;
    if ((a->q_indptr != nullptr) != ctx->plan_ragged) return NSD_ERR_INVALID_ARG;   // the plan fixed the rows' layout
    const int64_t rows = ctx->plan_rows;
    const int64_t kv_layer = rows * Hkv * D, q_layer = rows * Hq * D;
    const int64_t* qi = a->q_indptr;
    const uint16_t* k_new = static_cast<const uint16_t*>(a->k_new);
    const uint16_t* v_new = static_cast<const uint16_t*>(a->v_new);
    const uint16_t* q = static_cast<const uint16_t*>(a->q);
    uint16_t* o = static_cast<uint16_t*>(a->o);

    const int64_t n_pairs = a->n_mig_blocks;
    if (a->fuse_gather != 0 && a->fuse_gather != 1) return NSD_ERR_INVALID_ARG;
    if (a->fuse_gather && n_pairs != ctx->plan_src_blocks) return NSD_ERR_INVALID_ARG;   // the plan walks the same list
    const bool fused = a->fuse_gather && n_pairs > 0;
    const bool overlap = n_pairs > 0 && !fused;
    // The first layer has nothing to hide its copy behind but itself: its resident requests can be appended and
    // attended while the copy runs, the reassigned ones after it.  That costs a second, partial attention launch
    // (tens of microseconds of ramp and tail), so it only pays when the copy is longer than that: from about
    // 60 us of copying (384 MiB read + written) on.  Below, the layer simply waits for its copy.
    const int64_t copy_bytes = n_pairs * ctx->shape.block_elems() * 2 * (int64_t)sizeof(uint16_t);
    // The split needs the plan's resident / reassigned item lists: a plan made without is_migrated has every request
    // on the resident list, and attending that list before the copy event would read blocks still being written.
    const bool can_split = ctx->plan_has_mig && ctx->n_mig_items > 0 && ctx->plan_src_blocks == n_pairs;
    const bool split_first = can_split && (ctx->round_split == 1 || (ctx->round_split == 0 && copy_bytes >= (384LL << 20)));
    // A first layer that waits for its copy anyway runs the copy on the caller's stream: no event hop.
    const bool first_copy_inline = overlap && !split_first;
    if (overlap && (L > 1 || !first_copy_inline)) {
        NSD_CUDA(ctx, cudaEventRecord(ctx->ev_start, st));
        NSD_CUDA(ctx, cudaStreamWaitEvent(ctx->side, ctx->ev_start, 0));
    }
    // Kernels of this round that follow a kernel of this round on the caller's stream are launched as its programmatic
    // dependents: each reads its own inputs and sets itself up beside the tail of the one before, and waits
    // (griddepcontrol.wait) before it touches the pool or writes an output.
    bool chained = false;
    auto dep = [&]() {
        const bool d = ctx->pdl && chained;
        chained = true;
        return d;
    };
    for (int l = 0; l < L; ++l) {
        uint16_t* slab = slab_ptr(ctx, a->kv_pool, l);
        if (hook) NSD_CUDA(ctx, cudaStreamWaitEvent(st, ctx->ev_in[l], 0));
        if (overlap) {
            // Side stream: the copy of layer l's blocks.  It needs nothing this round computes (the copied entries
            // were committed before the round), so it runs ahead of the main stream -- as many layers as there are
            // spare slabs -- and the copy of layer l + 1 is under way while layer l attends: Run || Prepare, layer by
            // layer.  The new tokens' rows, which a model only has once it reaches the layer, are appended on the
            // main stream, for every request, right before the layer's attention.
            const bool copy_inline = l == 0 && first_copy_inline;
            if (copy_inline) {
                NSD_CUDA(ctx, launch_gather(ctx->shape, slab, n_pairs, a->mig_src, a->mig_dst, ctx->d_status, ctx->n_sms, ctx->wait_budget, ctx->starve_gather, st));
                chained = true;
            } else {
                if (l >= S) NSD_CUDA(ctx, cudaStreamWaitEvent(ctx->side, ctx->ev_attn[l - S], 0));
                NSD_CUDA(ctx, launch_gather(ctx->shape, slab, n_pairs, a->mig_src, a->mig_dst, ctx->d_status, ctx->n_sms, ctx->wait_budget, ctx->starve_gather, ctx->side));
                NSD_CUDA(ctx, cudaEventRecord(ctx->ev_prep[l], ctx->side));
            }
            ctx->launches++;
            nsd_status s;
            if (l == 0 && split_first) {
                // nothing to hide the first copy behind but the first layer itself: its resident requests go first
                NSD_CUDA(ctx, launch_append(ctx->shape, slab, batch, gamma, qi, a->ctx_len, a->kv_indptr, a->kv_indices, k_new, v_new,
                                            a->is_migrated, 1, ctx->d_status, st, dep()));
                s = attn_enqueue(ctx, a->kv_pool, q, o, nullptr, gamma, a->ctx_len, a->kv_indptr, a->kv_indices, 0, 1, st, nullptr, dep());
                if (s != NSD_OK) return s;
                NSD_CUDA(ctx, cudaStreamWaitEvent(st, ctx->ev_prep[0], 0));
                NSD_CUDA(ctx, launch_append(ctx->shape, slab, batch, gamma, qi, a->ctx_len, a->kv_indptr, a->kv_indices, k_new, v_new,
                                            a->is_migrated, 2, ctx->d_status, st, dep()));
                s = attn_enqueue(ctx, a->kv_pool, q, o, nullptr, gamma, a->ctx_len, a->kv_indptr, a->kv_indices, 0, 2, st, nullptr, dep());
                ctx->launches += 2;
            } else {
                if (!copy_inline) NSD_CUDA(ctx, cudaStreamWaitEvent(st, ctx->ev_prep[l], 0));
                NSD_CUDA(ctx, launch_append(ctx->shape, slab, batch, gamma, qi, a->ctx_len, a->kv_indptr, a->kv_indices,
                                            k_new + l * kv_layer, v_new + l * kv_layer, nullptr, 0, ctx->d_status, st, dep()));
                s = attn_enqueue(ctx, a->kv_pool, q + l * q_layer, o + l * q_layer, nullptr, gamma, a->ctx_len,
                                 a->kv_indptr, a->kv_indices, l, 0, st, nullptr, dep());
                ctx->launches++;
            }
            if (s != NSD_OK) return s;
            if (l + S < L) NSD_CUDA(ctx, cudaEventRecord(ctx->ev_attn[l], st));
        } else if (fused) {
            // gather-through: only the resident requests are appended by the copy kernels; attention itself
            // moves the reassigned requests' blocks and new tokens while it streams them
            NSD_CUDA(ctx, launch_append(ctx->shape, slab, batch, gamma, qi, a->ctx_len, a->kv_indptr, a->kv_indices,
                                        k_new + l * kv_layer, v_new + l * kv_layer, a->is_migrated, 1, ctx->d_status, st, dep()));
            ctx->launches++;
            const FuseArgs f{a->mig_src, k_new + l * kv_layer, v_new + l * kv_layer};
            nsd_status s = attn_enqueue(ctx, a->kv_pool, q + l * q_layer, o + l * q_layer, nullptr, gamma, a->ctx_len,
                                        a->kv_indptr, a->kv_indices, l, 0, st, &f, dep());
            if (s != NSD_OK) return s;
        } else {
            NSD_CUDA(ctx, launch_append(ctx->shape, slab, batch, gamma, qi, a->ctx_len, a->kv_indptr, a->kv_indices,
                                        k_new + l * kv_layer, v_new + l * kv_layer, nullptr, 0, ctx->d_status, st, dep()));
            ctx->launches++;
            nsd_status s = attn_enqueue(ctx, a->kv_pool, q + l * q_layer, o + l * q_layer, nullptr, gamma, a->ctx_len,
                                        a->kv_indptr, a->kv_indices, l, 0, st, nullptr, dep());
            if (s != NSD_OK) return s;
        }
        if (hook) {
            NSD_CUDA(ctx, cudaEventRecord(ctx->ev_out[l], st));
            NSD_CUDA(ctx, cudaStreamWaitEvent(ctx->down, ctx->ev_out[l], 0));
            NSD_CUDA(ctx, cudaMemcpyAsync(static_cast<char*>(hook->h_o) + (size_t)l * hook->o_layer_bytes, o + l * q_layer,
                                          hook->o_layer_bytes, cudaMemcpyDeviceToHost, ctx->down));
        }
    }
    if (hook) {
        NSD_CUDA(ctx, cudaEventRecord(ctx->ev_down_done, ctx->down));
        NSD_CUDA(ctx, cudaStreamWaitEvent(st, hook->inputs_ready, 0));
    }
    NSD_CUDA(ctx, launch_accept(a->p, a->q_draft, a->draft_tok, a->u_acc, a->u_smp, batch, gamma, ctx->cfg.vocab_size, qi,
                                a->ctx_len, a->acc_len, a->out_tok, a->new_ctx_len, ctx->d_status, ctx->accept_split, st,
                                hook ? false : dep()));
    ctx->launches++;
    if (hook) NSD_CUDA(ctx, cudaStreamWaitEvent(st, ctx->ev_down_done, 0));      // the caller's stream covers the read-back
    return NSD_OK;
}
}  // namespace

nsd_status nsd_verify_round_host(nsd_ctx* ctx, const nsd_round_args* h, const nsd_round_args* d,
                                 int64_t total_table_entries, void* stream, int64_t* h2d_bytes,
                                 int64_t* d2h_bytes) {
    if (!ctx || !h || !d) return NSD_ERR_INVALID_ARG;
    const int32_t batch = h->batch, gamma = h->gamma;
    if (batch != d->batch || gamma != d->gamma || h->n_mig_blocks != d->n_mig_blocks || h->fuse_gather != d->fuse_gather) return NSD_ERR_INVALID_ARG;
    if (batch < 0 || batch > ctx->cfg.max_batch || gamma < 1 || gamma > ctx->cfg.max_gamma) return NSD_ERR_OUT_OF_RANGE;
    if (total_table_entries < 0 || total_table_entries > ctx->cfg.max_table_entries || h->n_mig_blocks < 0) return NSD_ERR_INVALID_ARG;
    if (batch == 0) return NSD_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int L = ctx->cfg.num_layers, Hq = ctx->cfg.num_q_heads, Hkv = ctx->cfg.num_kv_heads, D = ctx->cfg.head_dim;
    if ((h->q_indptr != nullptr) != (d->q_indptr != nullptr)) return NSD_ERR_INVALID_ARG;
    // ragged rows: the host copy of q_indptr gives the totals (target rows; one draft row fewer per request)
    const int64_t V = ctx->cfg.vocab_size, rows = h->q_indptr ? h->q_indptr[batch] : (int64_t)batch * (gamma + 1);
    if (rows < batch || rows > (int64_t)batch * (gamma + 1)) return NSD_ERR_INVALID_ARG;
    const int64_t drafts = rows - batch;
    int64_t up = 0, down = 0;
    struct Copy { const void* src; const void* dst; int64_t bytes; };
    // Everything goes up on the copy stream in the order it is needed: the tables, then layer by layer the new K / V
    // rows and the queries (each layer starts as soon as its own inputs have landed), then the acceptance inputs,
    // which travel while the layers run.  The output comes back layer by layer on a third stream.
    const int64_t kv_layer_bytes = rows * Hkv * D * 2, q_layer_bytes = rows * Hq * D * 2;
    const Copy tables[] = {
        {h->ctx_len, d->ctx_len, batch * 4LL},
        {h->kv_indptr, d->kv_indptr, (batch + 1) * 8LL},
        {h->kv_indices, d->kv_indices, total_table_entries * 4},
        {h->is_migrated, d->is_migrated, h->is_migrated ? batch * 1LL : 0},
        {h->mig_src, d->mig_src, h->n_mig_blocks * 4},
        {h->mig_dst, d->mig_dst, h->n_mig_blocks * 4},
        {h->q_indptr, d->q_indptr, h->q_indptr ? (batch + 1) * 8LL : 0},
    };
    // The probability tensors are by far the largest inputs (2.8 GB at batch 512 and the Qwen3 vocabulary), yet the
    // acceptance reads gamma scalars and one row (pair) per request of them.  Where the caller's buffers are pinned host
    // memory that the device can address, they are not copied: the acceptance kernel reads what it needs over the link.
    auto device_view = [](const void* hp) -> const void* {
        cudaPointerAttributes at{};
        if (!hp || cudaPointerGetAttributes(&at, hp) != cudaSuccess) {
            cudaGetLastError();
            return nullptr;
        }
        return at.type == cudaMemoryTypeHost ? at.devicePointer : nullptr;
    };
    const float* p_direct = static_cast<const float*>(device_view(h->p));
    const float* q_direct = static_cast<const float*>(device_view(h->q_draft));
    const bool direct = p_direct && q_direct;
    const Copy accept_in[] = {
        {h->p, d->p, direct ? 0 : rows * V * 4},
        {h->q_draft, d->q_draft, direct ? 0 : drafts * V * 4},
        {h->draft_tok, d->draft_tok, drafts * 4},
        {h->u_acc, d->u_acc, drafts * 4},
        {h->u_smp, d->u_smp, batch * 4LL},
    };
    for (const Copy& c : tables)
        if (c.bytes != 0 && (!c.src || !c.dst)) return NSD_ERR_INVALID_ARG;
    for (const Copy& c : accept_in)
        if (c.bytes != 0 && (!c.src || !c.dst)) return NSD_ERR_INVALID_ARG;
    if (!h->p || !h->q_draft || (!direct && (!d->p || !d->q_draft))) return NSD_ERR_INVALID_ARG;
    if (!h->k_new || !d->k_new || !h->v_new || !d->v_new || !h->q || !d->q) return NSD_ERR_INVALID_ARG;
    if (!h->o || !d->o || !h->acc_len || !d->acc_len || !h->out_tok || !d->out_tok) return NSD_ERR_INVALID_ARG;
    nsd_status s = nsd_verify_plan(ctx, batch, gamma, h->ctx_len, h->kv_indptr, h->is_migrated, h->q_indptr, 0, stream);
    if (s != NSD_OK) return s;
    NSD_CUDA(ctx, cudaEventRecord(ctx->ev_copy_go, st));          // the device buffers are free once prior work is done
    NSD_CUDA(ctx, cudaStreamWaitEvent(ctx->copy, ctx->ev_copy_go, 0));
    NSD_CUDA(ctx, cudaStreamWaitEvent(ctx->down, ctx->ev_copy_go, 0));
    auto upload = [&](const Copy& c) -> cudaError_t {
        if (c.bytes == 0) return cudaSuccess;
        up += c.bytes;
        return cudaMemcpyAsync(const_cast<void*>(c.dst), c.src, (size_t)c.bytes, cudaMemcpyHostToDevice, ctx->copy);
    };
    for (const Copy& c : tables) NSD_CUDA(ctx, upload(c));
    NSD_CUDA(ctx, cudaEventRecord(ctx->ev_tables, ctx->copy));
    NSD_CUDA(ctx, cudaStreamWaitEvent(st, ctx->ev_tables, 0));
    for (int l = 0; l < L; ++l) {
        NSD_CUDA(ctx, upload({static_cast<const char*>(h->k_new) + l * kv_layer_bytes, static_cast<const char*>(d->k_new) + l * kv_layer_bytes, kv_layer_bytes}));
        NSD_CUDA(ctx, upload({static_cast<const char*>(h->v_new) + l * kv_layer_bytes, static_cast<const char*>(d->v_new) + l * kv_layer_bytes, kv_layer_bytes}));
        NSD_CUDA(ctx, upload({static_cast<const char*>(h->q) + l * q_layer_bytes, static_cast<const char*>(d->q) + l * q_layer_bytes, q_layer_bytes}));
        NSD_CUDA(ctx, cudaEventRecord(ctx->ev_in[l], ctx->copy));
    }
    for (const Copy& c : accept_in) NSD_CUDA(ctx, upload(c));
    NSD_CUDA(ctx, cudaEventRecord(ctx->ev_accept_in, ctx->copy));
    const BeforeAccept hook{h->o, (size_t)q_layer_bytes, ctx->ev_accept_in};
    nsd_round_args dd = *d;
    if (direct) {
        dd.p = p_direct;
        dd.q_draft = q_direct;
    }
    s = round_impl(ctx, &dd, stream, &hook);
    if (s != NSD_OK) {
        cudaStreamSynchronize(ctx->copy);
        cudaStreamSynchronize(ctx->down);
        return s;
    }
    down += (int64_t)hook.o_layer_bytes * L;
    const Copy downs[] = {
        {d->acc_len, h->acc_len, batch * 4LL},
        {d->out_tok, h->out_tok, rows * 4},
        {d->new_ctx_len, h->new_ctx_len, (d->new_ctx_len && h->new_ctx_len) ? batch * 4LL : 0},
    };
    for (const Copy& c : downs) {
        if (c.bytes == 0) continue;
        NSD_CUDA(ctx, cudaMemcpyAsync(const_cast<void*>(c.dst), c.src, (size_t)c.bytes, cudaMemcpyDeviceToHost, st));
        down += c.bytes;
    }
    NSD_CUDA(ctx, cudaStreamSynchronize(st));
    if (direct) {
        // what the acceptance kernel read over the link: per request the gathers of its tests and the one row (pair) of the draw
        for (int r = 0; r < batch; ++r) {
            const int64_t g_r = h->q_indptr ? h->q_indptr[r + 1] - h->q_indptr[r] - 1 : gamma;
            const int64_t n = h->acc_len[r];
            up += (n < g_r ? 2 : 1) * V * 4 + 2 * 4 * std::min<int64_t>(g_r, n + 1);
        }
    }
    if (h2d_bytes) *h2d_bytes = up;
    if (d2h_bytes) *d2h_bytes = down;
    return NSD_OK;
}

int64_t nsd_launch_count(const nsd_ctx* ctx) { return ctx ? ctx->launches : 0; }

nsd_status nsd_get_status(nsd_ctx* ctx, void* stream, int32_t* first_bad_request) {
    if (!ctx) return NSD_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    NSD_CUDA(ctx, cudaStreamSynchronize(ctx->side));
    NSD_CUDA(ctx, cudaMemcpyAsync(ctx->h_status, ctx->d_status, 4 * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    NSD_CUDA(ctx, cudaMemsetAsync(ctx->d_status, 0, 4 * sizeof(int32_t), st));
    NSD_CUDA(ctx, cudaStreamSynchronize(st));
    if (first_bad_request) *first_bad_request = ctx->h_status[1] - 1;
    if (ctx->h_status[0] & STATUS_TIMEOUT) {
        // A CTA that gave up never arrived at its request's split-KV counter, so the counter did not return to zero:
        // clear the arrival counters (attention and acceptance) so that the next launch starts clean.
        const Layout L = make_layout(&ctx->cfg);
        NSD_CUDA(ctx, cudaMemsetAsync(ctx->ws + L.counters, 0, L.items_all - L.counters, st));
        NSD_CUDA(ctx, cudaStreamSynchronize(st));
        return NSD_ERR_TIMEOUT;
    }
    if (ctx->h_status[0] & STATUS_LAYOUT) return NSD_ERR_UNSUPPORTED;     // the tcgen05 kernel found its shared memory unaligned
    return ctx->h_status[0] ? NSD_ERR_DEVICE_FAULT : NSD_OK;
}

}  // extern "C"
