// CPU oracle for the target-side verification round of M-for-N speculative decoding.
//
// TEST INFRASTRUCTURE, NOT PRODUCT.  Only the tests, the smoke check and the
// benchmark's cpu_baseline / reference arm may build, load or call this file.
// It shares no code, header, table or constant with the CUDA library: it is
// written from the definitions alone, slow and plain on purpose (double
// accumulators, two-pass softmax, sequential CDF, memcpy block copies, no
// tiling, no online softmax).  The only parallelism is a thread pool over
// independent requests, which changes no arithmetic.
//
// What each function follows:
//  * oracle_kv_prepare  -- Section 3 "KV cache organization" (paged KV, block
//    maps, append-dominant state) and Appendix E.2 (two banks with separate
//    block ranges; state must be present in the destination bank before Run,
//    Eq. (F.3)).  The result is its own definition: whole-block copies from
//    source to destination ids, then the new tokens written through the table.
//  * oracle_kv_commit   -- Section 5 "Incremental KV writeback" and Eq. (9): only the
//    committed suffix of each request moves to the export copy.
//  * oracle_verify_attn -- Section 1 / Appendix G.2: the target processes the
//    anchor token plus gamma proposal tokens of each request in one pass; the
//    attention itself is the textbook softmax(q K^T / sqrt(d)) V, causal among
//    the new tokens, grouped-query head mapping h -> h div (Hq/Hkv).
//  * oracle_spec_accept -- Section 1 cites the standard speculative-sampling
//    rule (Leviathan et al. 2023; Chen et al. 2023): accept draft i while
//    u_i < min(1, p_i(x_i)/q_i(x_i)); at the first rejection draw from the
//    normalised residual max(0, p - q); if nothing is rejected draw a bonus
//    token from the next target row.  Draws are inverse-CDF over token ids.
//
// Parity pins (tests/test_oracle_*.py): hand-worked V=4 example, closed-form
// acceptance statistics, chi-square of the committed-token law with a negative
// control, numpy brute force, K=0 / equal-V closed forms, permutation
// invariance and torch scaled_dot_product_attention on gathered KV.
#include <atomic>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <functional>
#include <limits>
#include <thread>
#include <vector>

namespace {

inline double bf16_to_double(uint16_t bits) {
    uint32_t u = static_cast<uint32_t>(bits) << 16;
    float f;
    std::memcpy(&f, &u, sizeof f);
    return static_cast<double>(f);
}

// Runs fn(i) for i in [0, n) on `nthreads` threads (dynamic assignment).
void parallel_for(int64_t n, int nthreads, const std::function<void(int64_t)>& fn) {
    if (nthreads <= 1 || n <= 1) {
        for (int64_t i = 0; i < n; ++i) fn(i);
        return;
    }
    std::atomic<int64_t> next{0};
    std::vector<std::thread> pool;
    int nt = static_cast<int>(std::min<int64_t>(nthreads, n));
    for (int t = 0; t < nt; ++t)
        pool.emplace_back([&] {
            for (;;) {
                int64_t i = next.fetch_add(1);
                if (i >= n) return;
                fn(i);
            }
        });
    for (auto& th : pool) th.join();
}

// Pool addressing: [slab][block][K|V][kv_head][slot][dim], bf16.
struct PoolShape {
    int64_t num_blocks;
    int Hkv, bs, D;
    int64_t block_elems() const { return 2LL * Hkv * bs * D; }
    int64_t slab_elems() const { return num_blocks * block_elems(); }
    int64_t at(int64_t slab, int64_t block, int kv, int head, int slot, int dim) const {
        return ((((slab * num_blocks + block) * 2 + kv) * Hkv + head) * bs + slot) * D + dim;
    }
};

// Rows per request when drafts are ragged (Appendix G.2 studies draft depths 3, 4, 5: the target verifies "anchor plus
// proposal" tokens of each request, and a batch may mix depths).  Request r brings gamma_r[r] proposals, so gamma_r[r] + 1
// rows; its rows start at the sum of the rows before it.  With gamma_r == nullptr every request has gamma + 1 rows.
// Returns false when a depth lies outside [0, gamma].
bool row_offsets(int batch, int gamma, const int32_t* gamma_r, std::vector<int64_t>& row0, std::vector<int>& depth) {
    row0.assign(batch + 1, 0);
    depth.assign(batch, gamma);
    for (int r = 0; r < batch; ++r) {
        if (gamma_r) {
            if (gamma_r[r] < 0 || gamma_r[r] > gamma) return false;
            depth[r] = gamma_r[r];
        }
        row0[r + 1] = row0[r] + depth[r] + 1;
    }
    return true;
}

}  // namespace

extern "C" {

int oracle_hardware_threads() {
    unsigned n = std::thread::hardware_concurrency();
    return n ? static_cast<int>(n) : 1;
}

// Gather, then append, one logical layer after the other.  Logical layer l
// lives in physical slab l % num_slabs.  k_new / v_new are indexed by logical
// layer: [num_layers][rows][Hkv][D]; pass nullptr to skip the append.  gamma_r
// (nullable): per-request draft depth, rows ragged (see row_offsets).
// Returns 0, or a negative code when an index leaves its range (nothing is
// written for that item).
int oracle_kv_prepare(uint16_t* pool, int num_slabs, int64_t num_blocks, int Hkv, int bs, int D,
                      int n_mig, const int64_t* mig_indptr, const int32_t* mig_src, const int32_t* mig_dst,
                      int batch, int gamma, const int32_t* ctx_len, const int64_t* kv_indptr,
                      const int32_t* kv_indices, const uint16_t* k_new, const uint16_t* v_new,
                      int layer_begin, int layer_count, const int32_t* gamma_r) {
    PoolShape ps{num_blocks, Hkv, bs, D};
    const int64_t blk = ps.block_elems();
    std::vector<int64_t> row0;
    std::vector<int> depth;
    if (!row_offsets(batch, gamma, gamma_r, row0, depth)) return -7;
    const int64_t layer_rows = row0[batch];
    int rc = 0;
    for (int l = layer_begin; l < layer_begin + layer_count; ++l) {
        const int64_t slab = l % num_slabs;
        uint16_t* base = pool + slab * ps.slab_elems();
        // gather: whole blocks, tail slots included
        for (int m = 0; m < n_mig; ++m)
            for (int64_t e = mig_indptr[m]; e < mig_indptr[m + 1]; ++e) {
                int64_t s = mig_src[e], d = mig_dst[e];
                if (s < 0 || s >= num_blocks || d < 0 || d >= num_blocks) { rc = -1; continue; }
                std::memcpy(base + d * blk, base + s * blk, static_cast<size_t>(blk) * sizeof(uint16_t));
            }
        if (!k_new || !v_new) continue;
        // append: token t of request r goes to position ctx_r + t
        for (int r = 0; r < batch; ++r)
            for (int t = 0; t <= depth[r]; ++t) {
                int64_t pos = static_cast<int64_t>(ctx_len[r]) + t;
                int64_t entry = kv_indptr[r] + pos / bs;
                if (ctx_len[r] < 0 || entry >= kv_indptr[r + 1]) { rc = -2; continue; }
                int64_t b = kv_indices[entry];
                if (b < 0 || b >= num_blocks) { rc = -1; continue; }
                int slot = static_cast<int>(pos % bs);
                int64_t row = static_cast<int64_t>(l) * layer_rows + row0[r] + t;
                for (int h = 0; h < Hkv; ++h) {
                    std::memcpy(pool + ps.at(slab, b, 0, h, slot, 0), k_new + (row * Hkv + h) * D, D * sizeof(uint16_t));
                    std::memcpy(pool + ps.at(slab, b, 1, h, slot, 0), v_new + (row * Hkv + h) * D, D * sizeof(uint16_t));
                }
            }
    }
    return rc;
}

// Suffix commit (Section 5, "Incremental KV writeback": only the KV suffix that is
// not yet persistent is written back, the prefix stays; cost Delta_Q * b_KV of
// Eq. (9)).  After acceptance, request r has committed its anchor and acc_len[r]
// drafts: positions ctx_r .. ctx_r + acc_len[r].  Each of them is copied, every kv
// head, K and V, from the block its table names to the block the export table names
// (same position -> same entry index and slot).  Rejected drafts are not copied.
int oracle_kv_commit(uint16_t* pool, int num_slabs, int64_t num_blocks, int Hkv, int bs, int D, int batch, int gamma,
                     const int32_t* ctx_len, const int32_t* acc_len, const int64_t* kv_indptr,
                     const int32_t* kv_indices, const int64_t* exp_indptr, const int32_t* exp_indices,
                     int32_t* new_ctx_len, int layer_begin, int layer_count, const int32_t* gamma_r) {
    PoolShape ps{num_blocks, Hkv, bs, D};
    int rc = 0;
    for (int l = layer_begin; l < layer_begin + layer_count; ++l) {
        const int64_t slab = l % num_slabs;
        for (int r = 0; r < batch; ++r) {
            if (acc_len[r] < 0 || acc_len[r] > (gamma_r ? gamma_r[r] : gamma)) { rc = -6; continue; }   // at most the drafts it had
            for (int t = 0; t <= acc_len[r]; ++t) {
                const int64_t pos = static_cast<int64_t>(ctx_len[r]) + t;
                const int64_t from = kv_indices[kv_indptr[r] + pos / bs], to = exp_indices[exp_indptr[r] + pos / bs];
                if (from < 0 || from >= num_blocks || to < 0 || to >= num_blocks) { rc = -1; continue; }
                const int slot = static_cast<int>(pos % bs);
                for (int kv = 0; kv < 2; ++kv)
                    for (int h = 0; h < Hkv; ++h)
                        std::memcpy(pool + ps.at(slab, to, kv, h, slot, 0), pool + ps.at(slab, from, kv, h, slot, 0), D * sizeof(uint16_t));
            }
        }
    }
    if (new_ctx_len)
        for (int r = 0; r < batch; ++r) new_ctx_len[r] = ctx_len[r] + 1 + acc_len[r];
    return rc;
}

// Attention of one logical layer.  q: [rows][Hq][D] bf16 for this layer;
// o: [rows][Hq][D] fp32; lse (nullable): [rows][Hq] natural-log sum-exp of the
// scaled scores.  Row i of request r sees keys [0, ctx_r + i].  When req_list
// is non-null only those requests are computed (others' outputs untouched).
int oracle_verify_attn(const uint16_t* pool, int num_slabs, int64_t num_blocks, int Hq, int Hkv, int bs, int D,
                       const uint16_t* q, float* o, float* lse, int batch, int gamma, const int32_t* ctx_len,
                       const int64_t* kv_indptr, const int32_t* kv_indices, int layer,
                       const int32_t* req_list, int n_req, int nthreads, const int32_t* gamma_r) {
    if (Hkv <= 0 || Hq % Hkv != 0) return -3;
    std::vector<int64_t> row0;
    std::vector<int> depth;
    if (!row_offsets(batch, gamma, gamma_r, row0, depth)) return -7;
    PoolShape ps{num_blocks, Hkv, bs, D};
    const int group = Hq / Hkv;
    const int64_t slab = layer % num_slabs;
    const double scale = 1.0 / std::sqrt(static_cast<double>(D));
    const int64_t n_items = req_list ? n_req : batch;
    std::atomic<int> rc{0};
    parallel_for(n_items, nthreads, [&](int64_t it) {
        const int r = req_list ? req_list[it] : static_cast<int>(it);
        if (r < 0 || r >= batch) { rc = -4; return; }
        std::vector<double> s, acc(D);
        for (int i = 0; i <= depth[r]; ++i) {
            const int64_t n_keys = static_cast<int64_t>(ctx_len[r]) + i + 1;
            const int64_t row = row0[r] + i;
            s.resize(n_keys);
            for (int h = 0; h < Hq; ++h) {
                const int g = h / group;
                const uint16_t* qv = q + (row * Hq + h) * D;
                double m = -std::numeric_limits<double>::infinity();
                for (int64_t j = 0; j < n_keys; ++j) {
                    int64_t b = kv_indices[kv_indptr[r] + j / bs];
                    const uint16_t* kv = pool + ps.at(slab, b, 0, g, static_cast<int>(j % bs), 0);
                    double dot = 0.0;
                    for (int d = 0; d < D; ++d) dot += bf16_to_double(qv[d]) * bf16_to_double(kv[d]);
                    s[j] = dot * scale;
                    if (s[j] > m) m = s[j];
                }
                double denom = 0.0;
                std::fill(acc.begin(), acc.end(), 0.0);
                for (int64_t j = 0; j < n_keys; ++j) {
                    double w = std::exp(s[j] - m);
                    denom += w;
                    int64_t b = kv_indices[kv_indptr[r] + j / bs];
                    const uint16_t* vv = pool + ps.at(slab, b, 1, g, static_cast<int>(j % bs), 0);
                    for (int d = 0; d < D; ++d) acc[d] += w * bf16_to_double(vv[d]);
                }
                float* ov = o + (row * Hq + h) * D;
                for (int d = 0; d < D; ++d) ov[d] = static_cast<float>(acc[d] / denom);
                if (lse) lse[row * Hq + h] = static_cast<float>(m + std::log(denom));
            }
        }
    });
    return rc;
}

// Acceptance.  p: [batch][gamma+1][V], q: [batch][gamma][V], fp32 -- or, with gamma_r
// (per-request draft depth), ragged: gamma_r[r] + 1 target rows, gamma_r[r] draft rows,
// draft tokens and accept uniforms, gamma_r[r] + 1 output tokens per request.  All
// compares and sums in double on the fp32 inputs; the residual p - q is an fp32
// subtraction, then widened.  out_tok: [batch][gamma+1] = accepted drafts, the
// resampled or bonus token, then -1 padding.
int oracle_spec_accept(const float* p, const float* q, const int32_t* draft_tok, const float* u_acc,
                       const float* u_smp, int batch, int gamma, int64_t vocab, const int32_t* ctx_len,
                       int32_t* acc_len, int32_t* out_tok, int32_t* new_ctx_len, int nthreads, const int32_t* gamma_r) {
    std::atomic<int> rc{0};
    std::vector<int64_t> row0;
    std::vector<int> depth;
    if (!row_offsets(batch, gamma, gamma_r, row0, depth)) return -7;
    parallel_for(batch, nthreads, [&](int64_t r) {
        // target rows start at row0[r]; the request has one draft row fewer than target rows, so its draft rows, draft
        // tokens and accept uniforms start at row0[r] - r
        const int gamma = depth[r];
        const int64_t d0 = row0[r] - r;
        const float* pr = p + row0[r] * vocab;
        const float* qr = q + d0 * vocab;
        const int32_t* draft_tok_r = draft_tok + d0;
        const float* u_acc_r = u_acc + d0;
        int n = gamma;
        for (int i = 0; i < gamma; ++i) {
            int32_t x = draft_tok_r[i];
            if (x < 0 || x >= vocab) { rc = -5; n = i; break; }
            double P = pr[i * vocab + x], Q = qr[i * vocab + x];
            double ratio = (Q > 0.0) ? P / Q : (P > 0.0 ? 1.0 : 0.0);
            double thr = ratio < 1.0 ? ratio : 1.0;
            if (!(static_cast<double>(u_acc_r[i]) < thr)) { n = i; break; }
        }
        const float* prow = pr + static_cast<int64_t>(n) * vocab;
        std::vector<double> w(vocab);
        double Z = 0.0;
        if (n < gamma) {
            const float* qrow = qr + static_cast<int64_t>(n) * vocab;
            for (int64_t k = 0; k < vocab; ++k) {
                float diff = prow[k] - qrow[k];          // fp32 subtraction
                w[k] = diff > 0.0f ? static_cast<double>(diff) : 0.0;
                Z += w[k];
            }
        }
        if (n == gamma || Z == 0.0) {                       // bonus row, or an empty residual
            Z = 0.0;
            for (int64_t k = 0; k < vocab; ++k) { w[k] = prow[k]; Z += w[k]; }
        }
        const double t = static_cast<double>(u_smp[r]) * Z;
        int64_t y = -1, last_pos = -1;
        double C = 0.0;
        for (int64_t k = 0; k < vocab; ++k) {
            C += w[k];
            if (w[k] > 0.0) last_pos = k;
            if (C > t) { y = k; break; }
        }
        if (y < 0) y = last_pos;
        acc_len[r] = n;
        int32_t* out = out_tok + row0[r];
        for (int i = 0; i <= gamma; ++i) out[i] = i < n ? draft_tok_r[i] : (i == n ? static_cast<int32_t>(y) : -1);
        if (new_ctx_len && ctx_len) new_ctx_len[r] = ctx_len[r] + 1 + n;
    });
    return rc;
}

// Acceptance straight from target logits (the step in front of oracle_spec_accept: the
// target's softmax with temperature is part of the rule, p_i = softmax(z_i / T)).
// logits: [batch][gamma+1][V] fp32 (bf16 callers widen exactly).  gamma_r (nullable):
// drafts actually proposed for request r (<= gamma); its bonus row is row gamma_r.
//   T > 0  p in double from the logits (max-subtracted, two passes), then exactly the rule
//          of oracle_spec_accept with every compare, the residual max(0, p - q) and the
//          sequential CDF in double.
//   T == 0 greedy verification: the target's token at position i is argmax_k z_i[k]
//          (smallest index on ties, NaN never wins); draft i is accepted iff it equals
//          it; the emitted token is the argmax of row n.  No uniforms, no q.
int oracle_spec_accept_logits(const float* logits, double temperature, const float* q, const int32_t* draft_tok,
                              const float* u_acc, const float* u_smp, int batch, int gamma, int64_t vocab,
                              const int32_t* gamma_r, const int32_t* ctx_len, int32_t* acc_len, int32_t* out_tok,
                              int32_t* new_ctx_len, int nthreads) {
    std::atomic<int> rc{0};
    parallel_for(batch, nthreads, [&](int64_t r) {
        const float* zr = logits + r * (gamma + 1) * vocab;
        const int g = gamma_r ? gamma_r[r] : gamma;
        int32_t* out = out_tok + r * (gamma + 1);
        for (int i = 0; i <= gamma; ++i) out[i] = -1;
        if (g < 0 || g > gamma) { rc = -7; acc_len[r] = 0; return; }
        auto argmax_row = [&](int i) {
            const float* z = zr + static_cast<int64_t>(i) * vocab;
            int64_t best = -1;
            for (int64_t k = 0; k < vocab; ++k)
                if (!(z[k] != z[k]) && (best < 0 || z[k] > z[best])) best = k;
            return best;
        };
        int n = g;
        int64_t y = -1;
        if (temperature == 0.0) {
            for (int i = 0; i < g; ++i)
                if (argmax_row(i) != draft_tok[r * gamma + i]) { n = i; break; }
            y = argmax_row(n);
        } else {
            std::vector<double> prob(vocab), w(vocab);
            auto softmax_row = [&](int i) {
                const float* z = zr + static_cast<int64_t>(i) * vocab;
                double m = -std::numeric_limits<double>::infinity();
                for (int64_t k = 0; k < vocab; ++k) if (z[k] > m) m = z[k];
                double sum = 0.0;
                for (int64_t k = 0; k < vocab; ++k) { prob[k] = std::exp((static_cast<double>(z[k]) - m) / temperature); sum += prob[k]; }
                for (int64_t k = 0; k < vocab; ++k) prob[k] /= sum;
            };
            const float* qr = q + r * gamma * vocab;
            for (int i = 0; i < g; ++i) {
                const int32_t x = draft_tok[r * gamma + i];
                if (x < 0 || x >= vocab) { rc = -5; n = i; break; }
                softmax_row(i);
                const double P = prob[x], Q = qr[i * vocab + x];
                const double ratio = (Q > 0.0) ? P / Q : (P > 0.0 ? 1.0 : 0.0);
                const double thr = ratio < 1.0 ? ratio : 1.0;
                if (!(static_cast<double>(u_acc[r * gamma + i]) < thr)) { n = i; break; }
            }
            softmax_row(n);
            double Z = 0.0;
            if (n < g) {
                const float* qrow = qr + static_cast<int64_t>(n) * vocab;
                for (int64_t k = 0; k < vocab; ++k) {
                    const double d = prob[k] - static_cast<double>(qrow[k]);
                    w[k] = d > 0.0 ? d : 0.0;
                    Z += w[k];
                }
            }
            if (n == g || Z == 0.0) {
                Z = 0.0;
                for (int64_t k = 0; k < vocab; ++k) { w[k] = prob[k]; Z += w[k]; }
            }
            const double t = static_cast<double>(u_smp[r]) * Z;
            int64_t last_pos = -1;
            double C = 0.0;
            for (int64_t k = 0; k < vocab; ++k) {
                C += w[k];
                if (w[k] > 0.0) last_pos = k;
                if (C > t) { y = k; break; }
            }
            if (y < 0) y = last_pos;
        }
        acc_len[r] = n;
        for (int i = 0; i < n; ++i) out[i] = draft_tok[r * gamma + i];
        out[n] = static_cast<int32_t>(y);
        if (new_ctx_len && ctx_len) new_ctx_len[r] = ctx_len[r] + 1 + n;
    });
    return rc;
}

}  // extern "C"
