// Worker-triggered batch reconstruction (Algorithm 1; Eq. (6) earliest predicted start,
// Eq. (7) service-admission bound, Eq. (8) admissibility; Appendix F.2 physical fit).
// Pure host code: it produces the batch membership that nsd_verify_plan and the round
// then consume.  See include/nsd.h for the contract and for the reading of the ranking.
#include <algorithm>
#include <cstdint>
#include <vector>

#include "nsd.h"

namespace {

struct Cand {
    int32_t idx;        // position in the caller's arrays
    double e;           // predecessor completion time available to the scheduler
    double s_single;    // Eq. (6) for the singleton batch {r}
    double d;           // Eq. (7)
};

}  // namespace

extern "C" nsd_status nsd_schedule_batch(const nsd_sched_params* prm, int32_t n, const uint8_t* eligible,
                                         const double* pred_done, const double* kv_ready, const int32_t* rows,
                                         const int32_t* blocks, const int32_t* tokens, int32_t* batch_out,
                                         int32_t* batch_size, double* batch_start) {
    if (!prm || !batch_size || n < 0) return NSD_ERR_INVALID_ARG;
    *batch_size = 0;
    if (batch_start) *batch_start = prm->worker_avail;
    if (n == 0) return NSD_OK;
    if (!pred_done || !kv_ready || !batch_out) return NSD_ERR_INVALID_ARG;
    if (prm->max_batch < 0 || prm->target_interval < 0 || prm->slack < 0) return NSD_ERR_INVALID_ARG;

    try {
    // candidate filter: eligible requests with their predicted readiness; a request must fit the worker on its own
    std::vector<Cand> cand;
    cand.reserve(n);
    for (int32_t i = 0; i < n; ++i) {
        if (eligible && !eligible[i]) continue;
        const int64_t ri = rows ? rows[i] : 1, bi = blocks ? blocks[i] : 0, ti = tokens ? tokens[i] : 0;
        if (ri < 0 || bi < 0 || ti < 0) return NSD_ERR_INVALID_ARG;
        if (ri > prm->row_capacity || bi > prm->block_capacity || ti > prm->token_limit) continue;
        Cand c;
        c.idx = i;
        c.e = pred_done[i];
        c.s_single = std::max(prm->worker_avail, std::max(pred_done[i], kv_ready[i]));
        c.d = std::max(pred_done[i] + prm->target_interval, c.s_single) + prm->slack;
        cand.push_back(c);
    }
    // sort key: urgency (admission bound), then predecessor readiness (older output first: the
    // waiting-time / aging component), then singleton start (temporal compatibility), then index
    std::stable_sort(cand.begin(), cand.end(), [](const Cand& a, const Cand& b) {
        if (a.d != b.d) return a.d < b.d;
        if (a.e != b.e) return a.e < b.e;
        if (a.s_single != b.s_single) return a.s_single < b.s_single;
        return a.idx < b.idx;
    });
    // only the first B_max candidates are considered
    if ((int64_t)cand.size() > prm->max_batch) cand.resize(prm->max_batch);

    // greedy admission in rank order under Eq. (8)
    double start = prm->worker_avail;     // Eq. (6) of the batch so far: max(a_w, max e, max k)
    double min_d = 0;
    int64_t used_rows = 0, used_blocks = 0, used_tokens = 0;
    int32_t m = 0;
    for (const Cand& c : cand) {
        const int64_t ri = rows ? rows[c.idx] : 1, bi = blocks ? blocks[c.idx] : 0, ti = tokens ? tokens[c.idx] : 0;
        const double new_start = std::max(start, c.s_single);
        const double new_min_d = m == 0 ? c.d : std::min(min_d, c.d);
        const bool fits = used_rows + ri <= prm->row_capacity && used_blocks + bi <= prm->block_capacity &&
                          used_tokens + ti <= prm->token_limit;
        if (m + 1 <= prm->max_batch && fits && new_start <= new_min_d) {
            batch_out[m++] = c.idx;
            start = new_start;
            min_d = new_min_d;
            used_rows += ri;
            used_blocks += bi;
            used_tokens += ti;
        }
    }
    *batch_size = m;
    if (batch_start) *batch_start = start;
    return NSD_OK;
    } catch (...) {                       // the candidate list could not be allocated: nothing crosses the C boundary
        *batch_size = 0;
        return NSD_ERR_CAPACITY;
    }
}
