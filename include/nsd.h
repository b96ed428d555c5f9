/*
 * nsd.h -- C ABI of the B200 verification round for M-for-N speculative decoding.
 *
 * One round = the target-side work on a batch that was rebuilt from the shared
 * request pool (Algorithm 1 hands it over as PREPARE followed by RUN):
 *   1. nsd_kv_prepare   make the KV state of every request present in this
 *                       worker's pool region, then append the new tokens' KV;
 *   2. nsd_verify_attn  ragged paged grouped-query attention, gamma+1 causal
 *                       query rows per request (anchor + gamma proposals);
 *   3. nsd_spec_accept  speculative acceptance / residual resampling / bonus.
 * nsd_verify_round enqueues all three for every layer, with the block copies on
 * a side stream that runs ahead of attention (Section 4: Run(B_k) || Prepare(B_k+1),
 * here layer by layer inside one batch: the copy of layer l+1 is under way while
 * layer l attends; only the first layer overlaps its own copy, by attending its
 * resident requests first).
 *
 * Conventions
 *  - Every function returns nsd_status; NSD_OK = 0.  Nothing throws.
 *  - Pointers are DEVICE pointers unless the name starts with h_ (host).
 *  - The caller owns every buffer, including the workspace the context lives
 *    on; the library allocates no device memory.  nsd_create additionally owns
 *    one CUDA side stream, a few events and a small pinned host staging area,
 *    released by nsd_destroy.
 *  - Device work is enqueued on the cudaStream_t passed as `stream` (cast to
 *    void*; 0 = legacy default stream) and the call returns after enqueue.
 *  - Host-visible arguments are validated before anything is launched; a
 *    failing call launches nothing.  Device-side index checks (block ids read
 *    from device tables) never fault: a bad id is replaced by block 0, the
 *    event is recorded in a status word, and nsd_get_status reports it.
 *  - A context is one worker: its workspace holds the plan, the split-KV partials,
 *    the acceptance scratch and the status word.  nsd_verify_attn, nsd_spec_accept,
 *    nsd_spec_accept_logits and nsd_verify_round(_host) on ONE context must not
 *    overlap one another on the GPU (enqueue them on one stream, or order the streams
 *    with events).  nsd_kv_prepare and nsd_kv_commit touch only the pool and the
 *    status word and may run on other streams beside them, as long as the caller
 *    orders the accesses to the same blocks.  Different contexts are independent.
 *    nsd_create also owns a copy stream and a read-back stream used only by
 *    nsd_verify_round_host.
 *  - bf16 tensors are raw 16-bit patterns.  Compiled for sm_100a only.
 *
 * KV pool layout (bf16):
 *     kv_pool[slab][block][kv][kv_head][slot][dim]
 *       slab    in [0, num_slabs)     logical layer l lives in slab l % num_slabs
 *       block   in [0, num_blocks)    ids < region_b_begin: region A (sources),
 *                                     the rest: region B (this worker's bank);
 *                                     Appendix E.2's separate block ranges
 *       kv      0 = K, 1 = V
 *       slot    in [0, block_size)    token position inside the block
 *   so one (slab, block) is one contiguous chunk of 2*Hkv*block_size*head_dim
 *   bf16 (64 KiB at the Qwen3-8B shape), and one (slab, block, kv, head) tile is
 *   one contiguous block_size*head_dim chunk (4 KiB).
 *   num_slabs == num_layers in production; a smaller num_slabs lets a
 *   benchmark run all logical layers over fewer physical slabs.
 *
 * Block tables: request r owns entries kv_indices[kv_indptr[r] .. kv_indptr[r+1]);
 * token position t of the request lives in block kv_indices[kv_indptr[r] + t /
 * block_size], slot t % block_size (Section 3, "KV cache organization").
 * ctx_len[r] counts the KV entries committed BEFORE the round; the round
 * appends gamma+1 entries at positions ctx_len[r] .. ctx_len[r]+gamma, and
 * query row i of the request sees keys [0, ctx_len[r] + i].
 *
 * Ragged rows (per-request draft depth).  The target verifies the anchor plus the
 * proposal tokens of each request (Appendix G.2), and the draft depth is a knob of
 * the draft side (the depth study runs 3, 4 and 5), so one batch may mix depths.
 * Every call that takes a `q_indptr` (int64 [batch+1], q_indptr[0] = 0) then works
 * on ragged row tensors: request r has gamma_r = q_indptr[r+1] - q_indptr[r] - 1
 * proposals (0 <= gamma_r <= gamma, the `gamma` argument being the upper bound), its
 * gamma_r + 1 query / new-token / target-probability rows start at row q_indptr[r]
 * of tensors with q_indptr[batch] rows in all, and its gamma_r draft rows, draft
 * tokens and accept uniforms start at q_indptr[r] - r (one fewer per request) of
 * tensors with q_indptr[batch] - batch entries.  No padded row is read, computed or
 * appended.  With q_indptr null every request has gamma proposals and the tensors
 * have the padded shapes given at each call.  A depth outside [0, gamma] met on the
 * device is skipped and reported by nsd_get_status as DEVICE_FAULT.
 */
#ifndef NSD_H_
#define NSD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    NSD_OK = 0,
    NSD_ERR_INVALID_ARG = 1,   /* null pointer, negative size, malformed host table          */
    NSD_ERR_OUT_OF_RANGE = 2,  /* gamma, batch, layer or vocab outside the configured limits */
    NSD_ERR_CAPACITY = 3,      /* workspace, table or partial-result capacity exceeded       */
    NSD_ERR_UNSUPPORTED = 4,   /* head_dim / block_size / group size this build has no kernel for */
    NSD_ERR_CUDA = 5,          /* a CUDA runtime call failed; see nsd_last_error             */
    NSD_ERR_DEVICE_FAULT = 6,  /* a kernel met an out-of-range index in a device table       */
    NSD_ERR_NOT_PLANNED = 7,   /* nsd_verify_attn / nsd_verify_round before nsd_verify_plan  */
    NSD_ERR_TIMEOUT = 8        /* a bounded wait inside a kernel ran out (reported by nsd_get_status) */
} nsd_status;

typedef struct nsd_ctx nsd_ctx;

typedef struct {
    int32_t num_layers;        /* logical layers of one round                            */
    int32_t num_slabs;         /* physical layer slabs in the pool, 1..num_layers        */
    int32_t num_q_heads;
    int32_t num_kv_heads;      /* divides num_q_heads                                    */
    int32_t head_dim;          /* 64 or 128                                              */
    int32_t block_size;        /* 16                                                     */
    int32_t num_blocks;        /* blocks per slab, both regions                          */
    int32_t region_b_begin;    /* blocks [0,begin) = region A, [begin,num_blocks) = B    */
    int32_t max_batch;
    int32_t max_gamma;         /* (num_q_heads/num_kv_heads)*(max_gamma+1) <= 64         */
    int32_t vocab_size;
    int32_t flags;             /* NSD_FLAG_* bits, 0 = the defaults                      */
    int64_t max_table_entries; /* upper bound of kv_indptr[batch]                        */
    int32_t wait_budget;       /* polls a kernel spends on one barrier before it gives up with
                                  NSD_ERR_TIMEOUT; 0 = the default (seconds)             */
    int32_t reserved;          /* 0                                                      */
} nsd_config;

/* nsd_config.flags: alternative kernels that compute the same results (comparison runs and
 * tests), and one test hook. */
enum {
    NSD_FLAG_ATTN_CP_ASYNC = 1 << 0,      /* attention: K/V tiles by cp.async for every shape (default: tensor
                                             copies where they are the faster feed)                            */
    NSD_FLAG_ATTN_TCGEN05 = 1 << 1,       /* attention: the tcgen05 engine for every shape it supports (default:
                                             only for the shapes where it is the faster one)                   */
    NSD_FLAG_ATTN_NO_TCGEN05 = 1 << 2,    /* attention: never the tcgen05 engine                               */
    NSD_FLAG_LOGITS_DIRECT = 1 << 3,      /* nsd_spec_accept_logits reads rows with direct loads               */
    NSD_FLAG_ROUND_SPLIT_ALWAYS = 1 << 4, /* first layer of a round: always attend the resident requests while
                                             the reassigned ones are still being copied ...                    */
    NSD_FLAG_ROUND_SPLIT_NEVER = 1 << 5,  /* ... or never (default: only when the copy is long enough to be
                                             worth a second launch)                                            */
    NSD_FLAG_NO_DEPENDENT_LAUNCH = 1 << 6, /* nsd_verify_round: every kernel starts only when the one before it on
                                             the stream has completed (default: the round's kernels are launched
                                             as programmatic dependents, so that one sets itself up beside the
                                             tail of the one before)                                           */
    NSD_FLAG_TEST_STARVE_GATHER = 1 << 30 /* test hook for the bounded waits: the gather arms every barrier with
                                             16 bytes more than its copy delivers, so each wait runs out after
                                             wait_budget polls and nsd_get_status returns NSD_ERR_TIMEOUT; the
                                             copies themselves still complete before the kernel returns        */
};

const char* nsd_status_string(nsd_status s);
/* Text of the last failing CUDA call made through `ctx` (empty string if none). */
const char* nsd_last_error(const nsd_ctx* ctx);

/* Bytes of device workspace nsd_create needs for `cfg` (0 if cfg is invalid),
 * and bytes of a pool with cfg->num_slabs slabs. */
size_t nsd_workspace_bytes(const nsd_config* cfg);
size_t nsd_kv_pool_bytes(const nsd_config* cfg);

/* Builds a context on caller-provided DEVICE memory `d_workspace` (256-byte
 * aligned, at least nsd_workspace_bytes(cfg), zero-filled by this call on the
 * legacy default stream, which is synchronised before return).  The device
 * current at this call owns the context.  cfg->flags selects alternative kernels
 * (NSD_FLAG_*); the library reads no environment variable. */
nsd_status nsd_create(const nsd_config* cfg, void* d_workspace, size_t workspace_bytes, nsd_ctx** out);
nsd_status nsd_destroy(nsd_ctx* ctx);

/*
 * Host-side planning for one batch (the scheduler knows the lengths: a frozen
 * batch carries membership and expected state versions, Appendix F.3).
 * Validates lengths and tables, cuts every request's key range into chunks
 * (split-KV), orders the chunks longest first and uploads the work lists on
 * `stream`.  Must precede nsd_verify_attn / nsd_verify_round for that batch.
 *   h_ctx_len      [batch]    committed KV entries, >= 0
 *   h_kv_indptr    [batch+1]  non-decreasing, entry count of request r must
 *                             cover ceil((ctx_len[r]+gamma+1)/block_size)
 *   h_is_migrated  [batch]    nullable; 1 = reassigned to this worker this
 *                             round (its KV arrives through the gather).  Must hold the
 *                             values of the round's device is_migrated.  A plan made
 *                             without it serves any round, but such a round cannot
 *                             overlap its first layer with its own copy (it waits for
 *                             the copy, then attends everybody) and cannot fuse_gather
 *   h_q_indptr     [batch+1]  nullable; per-request draft depth (see "Ragged rows" below): request
 *                             r brings h_q_indptr[r+1] - h_q_indptr[r] - 1 proposals, each depth in
 *                             [0, gamma]; h_q_indptr[0] = 0.  Null: every request has gamma proposals
 *   chunk_blocks   0 = choose; else the split-KV chunk length in blocks (even, <= 256)
 * Errors: INVALID_ARG (null, negative length, short table), OUT_OF_RANGE
 * (batch > max_batch, gamma outside [1,max_gamma]), CAPACITY (table entries or
 * split count beyond the workspace, or the host could not allocate the work list).
 * batch == 0 is a valid empty plan.
 */
nsd_status nsd_verify_plan(nsd_ctx* ctx, int32_t batch, int32_t gamma, const int32_t* h_ctx_len,
                           const int64_t* h_kv_indptr, const uint8_t* h_is_migrated, const int64_t* h_q_indptr,
                           int32_t chunk_blocks, void* stream);

/*
 * KV-state preparation (Section 3 "fragmented copies"; Section 5 / Appendix E.2:
 * the destination bank is filled before Run) for layers
 * [layer_begin, layer_begin+layer_count):
 *   gather  for j in [0, n_mig_blocks): whole block mig_src[j] -> block
 *           mig_dst[j] (tail slots included; sources are left untouched).  The
 *           list is the concatenation, over the reassigned requests, of their
 *           ceil(ctx_len/block_size) (source, destination) block pairs;
 *   append  K/V of token t of request r written at position ctx_len[r]+t
 *           through the block table (the append-dominant update of Section 3).
 * Per layer the gather is enqueued before the append.
 *   kv_pool     in/out
 *   mig_src / mig_dst  int32 [n_mig_blocks]; n_mig_blocks == 0 skips the
 *               gather (pointers may then be null)
 *   k_new,v_new bf16 [num_layers][batch*(gamma+1)][num_kv_heads][head_dim],
 *               indexed by logical layer; both null skips the append
 *   is_migrated nullable uint8 [batch]; append_subset: 0 = every request,
 *               1 = only requests with is_migrated == 0, 2 = only == 1
 *               (1 and 2 need is_migrated)
 *   q_indptr    nullable device int64 [batch+1]: ragged rows; total_rows =
 *               q_indptr[batch] as the host knows it (the rows of one layer of
 *               k_new / v_new; ignored when q_indptr is null)
 * Destination and append blocks must be unique per request, else the result is
 * undefined (not checked).  Errors: INVALID_ARG, OUT_OF_RANGE (layers, gamma,
 * batch).  A bad block id on the device is skipped and reported by
 * nsd_get_status as DEVICE_FAULT.
 */
nsd_status nsd_kv_prepare(nsd_ctx* ctx, void* kv_pool, int64_t n_mig_blocks,
                          const int32_t* mig_src, const int32_t* mig_dst, int32_t batch, int32_t gamma,
                          const int32_t* ctx_len, const int64_t* kv_indptr, const int32_t* kv_indices,
                          const void* k_new, const void* v_new, const uint8_t* is_migrated,
                          int32_t append_subset, int32_t layer_begin, int32_t layer_count, const int64_t* q_indptr,
                          int64_t total_rows, void* stream);

/*
 * Verification attention for one logical layer (Appendix G.2: the target
 * processes anchor + proposal tokens; attention itself is softmax(q K^T /
 * sqrt(head_dim)) V, q head h reading kv head h / (num_q_heads/num_kv_heads)).
 * Uses the batch last given to nsd_verify_plan; ctx_len / kv_indptr must hold
 * the same values on the device.
 *   q    bf16 [batch*(gamma+1)][num_q_heads][head_dim]   (this layer's rows; ragged when the plan
 *        was given h_q_indptr: [q_indptr[batch]] rows, request r's from row q_indptr[r])
 *   o    bf16 same shape (written for the requests of `subset`)
 *   lse  nullable fp32 [batch*(gamma+1)][num_q_heads], natural-log sum-exp
 *   subset  0 = all requests, 1 = resident only, 2 = reassigned only
 * bf16 inputs, fp32 accumulation, bf16 output.
 */
nsd_status nsd_verify_attn(nsd_ctx* ctx, const void* kv_pool, const void* q, void* o, float* lse,
                           int32_t batch, int32_t gamma, const int32_t* ctx_len, const int64_t* kv_indptr,
                           const int32_t* kv_indices, int32_t layer, int32_t subset, void* stream);

/*
 * Speculative acceptance (the rule Section 1 cites: Leviathan et al. 2023,
 * Chen et al. 2023).  For request r: accept draft i while
 * u_acc[r][i] < min(1, p[r][i][x_i] / q[r][i][x_i]) (strict; q == 0 accepts iff
 * p > 0), n = number accepted; if n < gamma draw y from max(0, p[r][n] - q[r][n])
 * (from p[r][n] itself if that residual is empty), else draw the bonus token
 * from p[r][gamma]; draws are inverse-CDF over token ids: smallest k whose
 * cumulative weight exceeds u_smp[r] * total.  Compares and sums are done in
 * fp64 on the fp32 inputs; the residual is an fp32 subtraction.
 *   p  fp32 [batch][gamma+1][vocab]   q  fp32 [batch][gamma][vocab]
 *   draft_tok int32 [batch][gamma]    u_acc fp32 [batch][gamma]   u_smp fp32 [batch]
 *   acc_len int32 [batch]             out_tok int32 [batch][gamma+1]: accepted
 *   drafts, then y, then -1 padding
 *   ctx_len / new_ctx_len  nullable pair: new_ctx_len[r] = ctx_len[r] + 1 + n
 *   q_indptr  nullable device int64 [batch+1]: ragged rows -- p [rows][vocab], q [rows - batch][vocab],
 *   draft_tok / u_acc [rows - batch], out_tok [rows], rows = q_indptr[batch]; a request without
 *   proposals emits the token drawn from its one target row
 * Errors: INVALID_ARG, OUT_OF_RANGE (gamma, batch, vocab < 1).  A draft token
 * outside [0, vocab) counts as rejected and is reported as DEVICE_FAULT.
 */
nsd_status nsd_spec_accept(nsd_ctx* ctx, const float* p, const float* q, const int32_t* draft_tok,
                           const float* u_acc, const float* u_smp, int32_t batch, int32_t gamma, int32_t vocab,
                           const int32_t* ctx_len, int32_t* acc_len, int32_t* out_tok, int32_t* new_ctx_len,
                           const int64_t* q_indptr, void* stream);

/*
 * Acceptance straight from the target's logits: the step in front of nsd_spec_accept
 * (the p of the cited rule is the target's softmax; with a temperature,
 * p_i = softmax(z_i / T)), fused so that p is never materialised.
 *   logits        [batch][gamma+1][vocab], logits_dtype 0 = fp32, 1 = bf16
 *   temperature   > 0: sample as nsd_spec_accept does, with p formed on the fly;
 *                 0: greedy verification -- draft i is accepted iff it equals
 *                 argmax_k z_i[k] (smallest index on ties, NaN never wins) and the
 *                 emitted token is the argmax of row n; q, u_acc, u_smp may be null
 *   gamma_r       nullable int32 [batch]: drafts actually proposed for request r
 *                 (0..gamma; tensors stay padded to gamma); its bonus row is row
 *                 gamma_r[r]; an impossible value is reported and treated as 0
 *   everything else as nsd_spec_accept.
 * Only rows 0..n of a request are read (the sweep stops at the first rejection).
 * Exponentials are fp32 (ex2.approx), sums and compares fp64: against an all-fp64
 * evaluation a decision can differ only within fp32 rounding of p at a decision or
 * CDF boundary; greedy mode is exact.  A row needs a finite maximum.
 * Errors: INVALID_ARG (null, negative or NaN temperature), OUT_OF_RANGE,
 * UNSUPPORTED (dtype).
 */
nsd_status nsd_spec_accept_logits(nsd_ctx* ctx, const void* logits, int32_t logits_dtype, float temperature,
                                  const float* q, const int32_t* draft_tok, const float* u_acc, const float* u_smp,
                                  int32_t batch, int32_t gamma, int32_t vocab, const int32_t* gamma_r,
                                  const int32_t* ctx_len, int32_t* acc_len, int32_t* out_tok, int32_t* new_ctx_len,
                                  void* stream);

/*
 * Suffix commit after the acceptance (Section 5, "Incremental KV writeback": only
 * the KV suffix that changed is written back, the persistent prefix stays; cost
 * model Eq. (9), Delta_Q tokens x bytes per token).  Request r committed its anchor
 * and acc_len[r] drafts, i.e. positions ctx_len[r] .. ctx_len[r]+acc_len[r]; for
 * layers [layer_begin, layer_begin+layer_count) each of these positions is copied,
 * K and V of every kv head, from the block kv_indices names to the block
 * exp_indices names for the same position (entry index position / block_size, same
 * slot).  Rejected drafts stay behind.  acc_len is read on the device, so the call
 * can be enqueued right behind nsd_spec_accept / nsd_verify_round.
 *   acc_len      int32 [batch], each in [0, gamma] -- in [0, gamma_r] with q_indptr (nullable
 *                device int64 [batch+1], ragged rows) -- else reported as DEVICE_FAULT
 *   exp_indptr / exp_indices   the export copy's table; entries that cannot hold
 *                a committed position are never read (may be -1)
 *   new_ctx_len  nullable int32 [batch]: ctx_len[r] + 1 + acc_len[r]
 * Errors: INVALID_ARG, OUT_OF_RANGE (batch, gamma, layers); bad block ids are
 * skipped and reported by nsd_get_status.
 */
nsd_status nsd_kv_commit(nsd_ctx* ctx, void* kv_pool, int32_t batch, int32_t gamma, const int32_t* ctx_len,
                         const int32_t* acc_len, const int64_t* kv_indptr, const int32_t* kv_indices,
                         const int64_t* exp_indptr, const int32_t* exp_indices, int32_t* new_ctx_len,
                         int32_t layer_begin, int32_t layer_count, const int64_t* q_indptr, void* stream);

/* Per-round tensors of nsd_verify_round; every pointer on the device. */
typedef struct {
    void* kv_pool;
    int64_t n_mig_blocks;         /* (source, destination) block pairs of the gather */
    const int32_t* mig_src;
    const int32_t* mig_dst;
    int32_t batch;
    int32_t gamma;
    const int32_t* ctx_len;
    const int64_t* kv_indptr;
    const int32_t* kv_indices;
    const uint8_t* is_migrated;   /* required when n_mig_blocks > 0 */
    const void* k_new;            /* [num_layers][rows][Hkv][D] */
    const void* v_new;
    const void* q;                /* [num_layers][rows][Hq][D]  */
    void* o;                      /* [num_layers][rows][Hq][D]  */
    const float* p;               /* acceptance inputs, as nsd_spec_accept */
    const float* q_draft;
    const int32_t* draft_tok;
    const float* u_acc;
    const float* u_smp;
    int32_t* acc_len;
    int32_t* out_tok;
    int32_t* new_ctx_len;         /* nullable */
    int32_t fuse_gather;          /* 0 = side-stream gather (default), 1 = gather-through attention */
    int32_t reserved;
    const int64_t* q_indptr;      /* nullable: ragged rows (the plan must have been given the same depths);
                                     every row tensor above then has q_indptr[batch] rows per layer,
                                     q_draft / draft_tok / u_acc q_indptr[batch] - batch entries */
} nsd_round_args;

/*
 * One whole verification round (every step above, every logical layer),
 * enqueued with the preparation overlapped behind attention: the side stream
 * copies the reassigned requests' blocks layer after layer, ahead of `stream`
 * (the copied entries were committed before the round); `stream` waits for a
 * layer's copy event (the KVReady condition of Eq. (F.3)), appends the new
 * tokens of every request and attends.  The first layer, which has nothing
 * else to hide its copy behind, appends and attends its resident requests
 * before that wait and the reassigned ones after it.  Acceptance follows the
 * last layer.  With num_slabs < num_layers the copy of layer l also waits for
 * the attention of layer l - num_slabs.  Needs a plan for this batch.  Returns
 * after enqueue; `stream` carries the completion.
 *
 * fuse_gather = 1 selects the gather-through variant (an extension beyond the
 * side-stream design; same pool bytes and outputs): there is no copy kernel and
 * no side stream; attention over a reassigned request reads its committed KV
 * from the SOURCE blocks, takes the new tokens from k_new / v_new, and writes
 * both into the destination blocks while it streams them, so the gather's read
 * disappears.  It needs the plan to have been given is_migrated, and mig_src to
 * list the reassigned requests' source blocks in request order,
 * ceil(ctx_len/block_size) entries each (INVALID_ARG if the counts disagree).
 */
nsd_status nsd_verify_round(nsd_ctx* ctx, const nsd_round_args* args, void* stream);

/*
 * The same round for a caller whose per-round tensors live in HOST memory
 * (pinned for full speed): every input of `h` except kv_pool is copied to the
 * matching buffer of `d` on `stream`, the round runs, and o, acc_len, out_tok
 * (and new_ctx_len when both are non-null) are copied back into `h`'s buffers;
 * the call synchronises `stream` before returning.  The acceptance inputs
 * (draft_tok, u_acc, u_smp) travel on an internal copy stream while the layers
 * run, and o is read back before the acceptance is enqueued, so the transfers
 * overlap the kernels.  p and q_draft, by far the largest inputs, are copied the
 * same way unless `h`'s buffers are pinned host memory the device can address
 * (cudaHostAlloc / cudaHostRegister): then they stay where they are and the
 * acceptance kernel reads the gamma scalars and the one row (pair) per request
 * it needs over the link (d->p, d->q_draft may then be null); the bytes it read
 * are counted in *h2d_bytes.  `h->kv_pool` is ignored:
 * the pool is worker state that stays on the device.  h_* table arguments of
 * the plan are taken from `h` (ctx_len, kv_indptr, is_migrated), so no separate
 * nsd_verify_plan call is needed.  Bytes moved are written to the two counters
 * when non-null.
 */
nsd_status nsd_verify_round_host(nsd_ctx* ctx, const nsd_round_args* h, const nsd_round_args* d,
                                 int64_t total_table_entries, void* stream, int64_t* h2d_bytes,
                                 int64_t* d2h_bytes);

/*
 * Attention for callers that are not allowed to allocate device memory.
 * (No counterpart in the paper: this entry point exists for the hosts of the
 * library, not for the method.)
 *
 * Who needs it: code that runs inside somebody else's memory budget (a plugin in
 * a serving runtime that owns the allocator), a worker whose device memory was
 * split up once at start-up and must not grow, or a latency path where an
 * allocator call may stall behind a device-wide synchronisation.  Such a caller
 * cannot provide the workspace nsd_create wants, so this variant of
 * nsd_verify_attn keeps its split-KV scratch (work list, arrival counters, fp32
 * partial results, status word) in a fixed array inside the library: about 8.1
 * MiB of device memory that every GPU loading the library holds until the
 * process exits.  The call itself performs no cudaMalloc / cudaFree and uses no
 * allocating library routine; it needs no nsd_ctx and no plan.
 *
 * Same result as nsd_verify_attn(subset = 0) for one layer slab:
 *   kv_slab     bf16 [num_blocks][2][num_kv_heads][block_size][head_dim] (one layer)
 *   q, o        bf16 [batch*(gamma+1)][num_q_heads][head_dim]
 *   h_ctx_len   HOST int32 [batch]  (used to cut the work list; must equal ctx_len)
 *   ctx_len, kv_indptr, kv_indices   device tables as for nsd_verify_attn; request r's
 *               table must cover ceil((h_ctx_len[r]+gamma+1)/block_size) entries.  This
 *               entry point has no host copy of kv_indptr to check that with: an entry
 *               index at or past kv_indptr[r+1] is not followed (block 0 is read instead)
 * Limits (NSD_ERR_CAPACITY beyond them, nothing launched): batch <= 64;
 * num_kv_heads <= 8; (num_q_heads/num_kv_heads)*(gamma+1) <= 32; requests longer
 * than 1024 keys are cut into 1024-key chunks and all such chunks of a call
 * together must number <= 64 (e.g. eight requests of 8K keys); work items
 * (chunks of all requests) <= 128.  head_dim 64 or 128, block_size 16
 * (NSD_ERR_UNSUPPORTED otherwise).  Other errors as nsd_verify_attn.
 *
 * The first call on a device resolves the array's address and sets kernel
 * attributes for that device.  No call of this entry point may be made while `stream`
 * is being captured into a CUDA graph: every call uploads its work list from a buffer
 * that lives only for the duration of the call (NSD_ERR_INVALID_ARG if the stream is
 * capturing).
 * All calls share the one array, and it keeps the previous call's contents: the
 * call clears the words that must start at zero, but two calls whose kernels can
 * overlap on the GPU (different streams, or the same call from two threads)
 * race on the scratch and give undefined results.  Serialise them.  Block ids
 * that are out of range are replaced by block 0; this variant does not report
 * them.
 */
nsd_status nsd_verify_attn_static(const void* kv_slab, int32_t num_blocks, int32_t num_q_heads,
                                  int32_t num_kv_heads, int32_t head_dim, int32_t block_size, const void* q,
                                  void* o, int32_t batch, int32_t gamma, const int32_t* h_ctx_len,
                                  const int32_t* ctx_len, const int64_t* kv_indptr, const int32_t* kv_indices,
                                  void* stream);

/*
 * Worker-triggered batch reconstruction on the host (Algorithm 1): which requests of
 * the stage's shared pool the triggered worker verifies next.  All times are seconds
 * on one clock.  For candidate r:
 *   S({r}) = max(worker_avail, pred_done[r], kv_ready[r])                    Eq. (6)
 *   d_r    = max(pred_done[r] + target_interval, S({r})) + slack             Eq. (7)
 * and a batch B is admissible (Eq. (8)) iff |B| <= max_batch, it fits the worker
 * (sum of rows / KV blocks / tokens within the capacities, Appendix F.2; a request
 * that does not fit alone is dropped), and S(B) = max over B of S({r}) <= min over B
 * of d_r.  Candidates are the `eligible` requests; they are ranked -- the paper names the
 * criteria (predecessor readiness, waiting time, temporal compatibility) but not the
 * key: this library sorts by d_r, then pred_done (older output first: the aging term),
 * then S({r}), then index --, the first max_batch of them are kept, and those are
 * admitted greedily in rank order while the batch stays admissible.  Freezing, PREPARE
 * and RUN are the caller's (nsd_verify_plan and nsd_verify_round take the chosen batch).
 *   eligible   nullable uint8 [n] (null = all); pred_done, kv_ready  double [n]
 *   rows / blocks / tokens   nullable int32 [n] (null = 1 row, 0 blocks, 0 tokens each)
 *   batch_out  int32 [min(n, max_batch)]: indices of the admitted requests in rank order
 *   batch_size, batch_start (nullable): |B| and S(B) (worker_avail for an empty batch)
 * Everything is host memory; nothing is launched.  Errors: INVALID_ARG.
 */
typedef struct {
    double worker_avail;      /* predicted availability of the triggered worker, a_w     */
    double target_interval;   /* g_s                                                     */
    double slack;             /* Delta_s                                                 */
    int32_t max_batch;        /* B_max                                                   */
    int32_t row_capacity;     /* batch rows the standby bank can take                    */
    int64_t block_capacity;   /* KV blocks it can take                                   */
    int64_t token_limit;      /* stage-specific token limit                              */
} nsd_sched_params;

nsd_status nsd_schedule_batch(const nsd_sched_params* prm, int32_t n, const uint8_t* eligible,
                              const double* pred_done, const double* kv_ready, const int32_t* rows,
                              const int32_t* blocks, const int32_t* tokens, int32_t* batch_out,
                              int32_t* batch_size, double* batch_start);

/* Number of kernels this library has launched through `ctx` since creation. */
int64_t nsd_launch_count(const nsd_ctx* ctx);

/* Synchronises the device work of `ctx` on `stream` and the side stream, then
 * reads the status word: NSD_OK, NSD_ERR_TIMEOUT (a copy never signalled its
 * barrier within the kernel's bounded wait), or NSD_ERR_DEVICE_FAULT with the first
 * offending request index (or -1) in *first_bad_request (nullable).  The word
 * is cleared by the call. */
nsd_status nsd_get_status(nsd_ctx* ctx, void* stream, int32_t* first_bad_request);

#ifdef __cplusplus
}
#endif
#endif /* NSD_H_ */
