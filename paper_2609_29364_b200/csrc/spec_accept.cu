// Speculative acceptance (the rule Section 1 cites from Leviathan et al. 2023 and
// Chen et al. 2023): accept draft i while u_i < min(1, p_i(x_i)/q_i(x_i)); at the
// first rejection draw from max(0, p - q); if nothing is rejected draw the bonus
// token from the next target row.
//
// One CTA per request.  Warp 0 decides the accepted length from gamma gathers;
// the whole CTA then sweeps ONLY the one vocabulary row pair that the draw needs
// (not all gamma+1), keeping one partial sum per 128-token segment in shared
// memory; the segment that holds the draw is found from the segment prefix and
// re-read (an L2 hit) to finish inside it.  When the batch is too small to fill
// the machine, `split` CTAs share a request: each sweeps its slice of the segments
// into a scratch row, and the last one to finish (atomic counter, nobody waits)
// collects the row and draws; segment sums, prefix and draw are the same numbers
// in the same order either way.  All compares and sums are fp64 on the
// fp32 inputs, the residual is a single fp32 subtraction, so decisions agree
// with a sequential fp64 evaluation except within rounding of a CDF boundary.
// Compile without fast-math: IEEE division and no flush-to-zero are required.
#include "nsd_internal.h"

namespace nsd {
namespace {

constexpr int kAcceptThreads = 512;
constexpr int kSeg = 128;                       // tokens per segment = one float4 per lane

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Weight of token k for the draw: residual (fp32 subtract, clamped) or the target row.
__device__ __forceinline__ float weight(float pv, float qv, bool residual) {
    if (!residual) return pv;
    const float d = __fsub_rn(pv, qv);
    return d > 0.0f ? d : 0.0f;
}

// Pass 1: one fp64 sum per 128-token segment of [s_begin, s_end), one warp per segment and pass.
// The destination is either the CTA's shared segment array (known address space: the loads of the next segment can
// be issued before the store of this one) or the request's scratch row in global memory.
template <bool RESIDUAL, bool TO_SHARED>
__device__ __forceinline__ void sweep_segments(const float* __restrict__ prow, const float* __restrict__ qrow, bool vec_ok,
                                               int vocab, int s_begin, int s_end, int warp, int lane,
                                               double* __restrict__ dst_global) {
    extern __shared__ double seg_sum_shared[];
    constexpr int n_warps = kAcceptThreads / 32;
    for (int s = s_begin + warp; s < s_end; s += n_warps) {
        const int k0 = s * kSeg + lane * 4;
        double acc = 0.0;
        if (vec_ok) {
            if (k0 < vocab) {
                const float4 pv = __ldg(reinterpret_cast<const float4*>(prow + k0));
                float4 qv = make_float4(0.f, 0.f, 0.f, 0.f);
                if (RESIDUAL) qv = __ldg(reinterpret_cast<const float4*>(qrow + k0));
                acc = (double)weight(pv.x, qv.x, RESIDUAL);
                acc += (double)weight(pv.y, qv.y, RESIDUAL);
                acc += (double)weight(pv.z, qv.z, RESIDUAL);
                acc += (double)weight(pv.w, qv.w, RESIDUAL);
            }
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (k0 + j < vocab) acc += (double)weight(prow[k0 + j], RESIDUAL ? qrow[k0 + j] : 0.f, RESIDUAL);
        }
        acc = warp_sum(acc);
        if (lane == 0) {
            if (TO_SHARED) seg_sum_shared[s] = acc;
            else dst_global[s] = acc;
        }
    }
}

struct AcceptArgs {
    const float* p;
    const float* q;
    const int32_t* draft_tok;
    const float* u_acc;
    const float* u_smp;
    int32_t gamma, vocab;
    const int64_t* q_indptr;     // nullable: ragged rows, request r has q_indptr[r+1] - q_indptr[r] - 1 drafts
    const int32_t* ctx_len;
    int32_t* acc_len;
    int32_t* out_tok;
    int32_t* new_ctx_len;
    int32_t* status;
    int32_t split;               // CTAs per request
    double* seg_scratch;
    int32_t* seg_counters;
};

// One body for both launch shapes.  SPLIT = several CTAs share a request (small batches): each sweeps its slice of
// the segments into the request's scratch row and the last to arrive (atomic counter, nobody waits) goes on alone.
template <bool SPLIT>
__device__ __forceinline__ void spec_accept_body(const AcceptArgs& a) {
    extern __shared__ double seg_sum[];          // [n_seg] segment sums, then exclusive prefixes
    __shared__ int s_n, s_found_seg, s_token, s_last;
    __shared__ double s_total;

    const int r = SPLIT ? blockIdx.x / a.split : blockIdx.x;
    const int part = SPLIT ? blockIdx.x - r * a.split : 0;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int vocab = a.vocab;
    const int n_seg = (vocab + kSeg - 1) / kSeg;
    // Rows of this request: padded ([batch][gamma+1] target rows, [batch][gamma] draft rows) or ragged (target rows from
    // q_indptr[r]; one draft row fewer per request, so draft rows, tokens and accept uniforms from q_indptr[r] - r).
    int gamma = a.gamma;
    int64_t row0 = (int64_t)r * (a.gamma + 1), d0 = (int64_t)r * a.gamma;
    if (a.q_indptr) {
        row0 = a.q_indptr[r];
        d0 = row0 - r;
        gamma = (int)(a.q_indptr[r + 1] - row0) - 1;
        if (gamma < 0 || gamma > a.gamma) {      // an impossible depth: reported, nothing of the request is read
            pdl_wait();
            if (tid == 0 && part == 0) {
                atomicOr(a.status, STATUS_BAD_TOKEN);
                atomicCAS(a.status + 1, 0, r + 1);
                a.acc_len[r] = 0;
            }
            if (SPLIT && tid == 0) {             // keep the arrival counter consistent
                const int old = atomicAdd(a.seg_counters + r, 1);
                if (old == a.split - 1) a.seg_counters[r] = 0;
            }
            return;
        }
    }
    const float* p_req = a.p + row0 * vocab;
    const float* q_req = a.q + d0 * vocab;
    const int32_t* tok_req = a.draft_tok + d0;

    // ---- accepted length: first i whose test fails
    if (warp == 0) {
        bool reject = false;
        if (lane < gamma) {
            const int32_t x = tok_req[lane];
            if ((uint32_t)x >= (uint32_t)vocab) {
                reject = true;
                atomicOr(a.status, STATUS_BAD_TOKEN);
                atomicCAS(a.status + 1, 0, r + 1);
            } else {
                const double P = (double)p_req[(int64_t)lane * vocab + x];
                const double Q = (double)q_req[(int64_t)lane * vocab + x];
                const double ratio = (Q > 0.0) ? P / Q : (P > 0.0 ? 1.0 : 0.0);
                const double thr = ratio < 1.0 ? ratio : 1.0;
                reject = !((double)a.u_acc[d0 + lane] < thr);
            }
        }
        const unsigned m = __ballot_sync(0xffffffffu, reject);
        if (lane == 0) s_n = m ? (__ffs(m) - 1) : gamma;
    }
    __syncthreads();
    // The tests above read the call's own inputs; the sweep and every output wait for the kernel before this one on
    // the stream (in a round: the last layer's attention, beside whose tail the tests ran).
    pdl_wait();
    const int n = s_n;
    const float* prow = p_req + (int64_t)n * vocab;
    const float* qrow = q_req + (int64_t)(n < gamma ? n : 0) * vocab;   // unused when n == gamma
    bool residual = n < gamma;
    const bool vec_ok = (vocab % 4 == 0) && ((reinterpret_cast<uintptr_t>(a.p) | reinterpret_cast<uintptr_t>(a.q)) % 16 == 0);

    // dst == nullptr: into seg_sum (shared); else into that global row
    auto sweep = [&](int s_begin, int s_end, double* dst, bool res) {
        if (dst == nullptr) {
            if (res) sweep_segments<true, true>(prow, qrow, vec_ok, vocab, s_begin, s_end, warp, lane, nullptr);
            else sweep_segments<false, true>(prow, qrow, vec_ok, vocab, s_begin, s_end, warp, lane, nullptr);
        } else {
            if (res) sweep_segments<true, false>(prow, qrow, vec_ok, vocab, s_begin, s_end, warp, lane, dst);
            else sweep_segments<false, false>(prow, qrow, vec_ok, vocab, s_begin, s_end, warp, lane, dst);
        }
    };
    // ---- exclusive prefix over segments (warp 0, lanes own consecutive runs)
    auto prefix = [&]() {
        if (warp == 0) {
            const int per = (n_seg + 31) / 32;
            const int b = lane * per, e = min(b + per, n_seg);
            double local = 0.0;
            for (int s = b; s < e; ++s) local += seg_sum[s];
            double incl = local;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const double up = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += up;
            }
            double run = incl - local;
            for (int s = b; s < e; ++s) {
                const double v = seg_sum[s];
                seg_sum[s] = run;
                run += v;
            }
            const double total = __shfl_sync(0xffffffffu, incl, 31);
            if (lane == 0) {
                s_total = total;
                s_found_seg = n_seg;
            }
        }
        __syncthreads();
    };

    if constexpr (SPLIT) {
        // this CTA's slice goes to the scratch row; whoever arrives last owns the rest of the work
        double* row = a.seg_scratch + (int64_t)r * n_seg;
        const int per = (n_seg + a.split - 1) / a.split;
        sweep(part * per, min((part + 1) * per, n_seg), row, residual);
        __threadfence();
        __syncthreads();
        if (tid == 0) {
            const int old = atomicAdd(a.seg_counters + r, 1);
            const int last = old == a.split - 1;
            if (last) a.seg_counters[r] = 0;         // ready for the next launch
            s_last = last;
        }
        __syncthreads();
        if (!s_last) return;
        __threadfence();
        for (int s = tid; s < n_seg; s += kAcceptThreads) seg_sum[s] = __ldcg(row + s);
        __syncthreads();
        prefix();
        if (residual && s_total == 0.0) {       // empty residual: draw from the target row instead
            residual = false;
            __syncthreads();
            sweep(0, n_seg, nullptr, false);
            __syncthreads();
            prefix();
        }
    } else {
        // one CTA owns the request: the sweep written out in place with `residual` a run-time flag (the templated
        // sweep costs this instantiation the 32 registers that let four CTAs share an SM)
        constexpr int n_warps = kAcceptThreads / 32;
        for (int attempt = 0; attempt < 2; ++attempt) {
            for (int s = warp; s < n_seg; s += n_warps) {
                const int k0 = s * kSeg + lane * 4;
                double acc = 0.0;
                if (vec_ok) {
                    if (k0 < vocab) {
                        const float4 pv = __ldg(reinterpret_cast<const float4*>(prow + k0));
                        float4 qv = make_float4(0.f, 0.f, 0.f, 0.f);
                        if (residual) qv = __ldg(reinterpret_cast<const float4*>(qrow + k0));
                        acc = (double)weight(pv.x, qv.x, residual);
                        acc += (double)weight(pv.y, qv.y, residual);
                        acc += (double)weight(pv.z, qv.z, residual);
                        acc += (double)weight(pv.w, qv.w, residual);
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        if (k0 + j < vocab) acc += (double)weight(prow[k0 + j], residual ? qrow[k0 + j] : 0.f, residual);
                }
                acc = warp_sum(acc);
                if (lane == 0) seg_sum[s] = acc;
            }
            __syncthreads();
            prefix();
            if (residual && s_total == 0.0) {   // empty residual: draw from the target row instead
                residual = false;
                __syncthreads();
                continue;
            }
            break;
        }
    }

    const double total = s_total;
    const double t = (double)a.u_smp[r] * total;
    // ---- first segment whose inclusive prefix exceeds t
    for (int s = tid; s < n_seg; s += kAcceptThreads) {
        const double incl = (s + 1 < n_seg) ? seg_sum[s + 1] : total;
        if (incl > t) {
            atomicMin(&s_found_seg, s);
            break;                               // a thread's later segments are larger
        }
    }
    __syncthreads();

    // ---- finish inside the segment (warp 0); walk on if rounding left nothing there
    if (warp == 0) {
        int token = -1;
        for (int s = s_found_seg; s < n_seg && token < 0; ++s) {
            const int k0 = s * kSeg + lane * 4;
            float w[4];
#pragma unroll
            for (int j = 0; j < 4; ++j)
                w[j] = (k0 + j < vocab) ? weight(prow[k0 + j], residual ? qrow[k0 + j] : 0.f, residual) : 0.f;
            const double mine = (double)w[0] + (double)w[1] + (double)w[2] + (double)w[3];
            double incl = mine;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const double up = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += up;
            }
            double c = seg_sum[s] + (incl - mine);
            int hit = -1;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                c += (double)w[j];
                if (hit < 0 && k0 + j < vocab && c > t) hit = k0 + j;
            }
            const unsigned m = __ballot_sync(0xffffffffu, hit >= 0);
            if (m) token = __shfl_sync(0xffffffffu, hit, __ffs(m) - 1);
        }
        if (token < 0 && lane == 0) {            // t not exceeded anywhere: last token with positive weight
            for (int k = vocab - 1; k >= 0; --k)
                if (weight(prow[k], residual ? qrow[k] : 0.f, residual) > 0.f) {
                    token = k;
                    break;
                }
        }
        if (lane == 0) s_token = token;
    }
    __syncthreads();

    if (tid <= gamma) {
        int32_t v = -1;
        if (tid < n) v = tok_req[tid];
        else if (tid == n) v = s_token;
        // (the row offset is read again rather than kept in registers across the sweep)
        a.out_tok[(a.q_indptr ? a.q_indptr[r] : (int64_t)r * (a.gamma + 1)) + tid] = v;
    }
    if (tid == 0) {
        a.acc_len[r] = n;
        if (a.new_ctx_len && a.ctx_len) a.new_ctx_len[r] = a.ctx_len[r] + 1 + n;
    }
}

// Four CTAs per SM (32 registers): at 40 registers only three fit and a full batch runs a quarter slower.
__global__ void __launch_bounds__(kAcceptThreads, 4) spec_accept_kernel(const __grid_constant__ AcceptArgs a) {
    spec_accept_body<false>(a);
}
// The same computation with `split` CTAs per request (small batches).
__global__ void __launch_bounds__(kAcceptThreads) spec_accept_split_kernel(const __grid_constant__ AcceptArgs a) {
    spec_accept_body<true>(a);
}

}  // namespace

cudaError_t launch_accept(const float* p, const float* q, const int32_t* draft_tok, const float* u_acc,
                          const float* u_smp, int32_t batch, int32_t gamma, int32_t vocab, const int64_t* q_indptr,
                          const int32_t* ctx_len, int32_t* acc_len, int32_t* out_tok, int32_t* new_ctx_len, int32_t* status,
                          const AcceptSplit& sp, cudaStream_t stream, bool pdl) {
    if (batch <= 0) return cudaSuccess;
    const int n_seg = (vocab + kSeg - 1) / kSeg;
    const size_t smem = (size_t)(n_seg + 1) * sizeof(double);
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(spec_accept_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(spec_accept_split_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    // Several CTAs per request while that still leaves the machine under two CTAs per SM, the slices at least
    // eight passes of a CTA long, and the scratch rows large enough.
    int split = 1;
    if (sp.scratch && sp.counters && batch <= sp.rows_cap && vocab <= sp.vocab_cap && sp.n_sms > 0) {
        split = (2 * sp.n_sms) / batch;
        split = split < 1 ? 1 : (split > 8 ? 8 : split);
        while (split > 1 && n_seg / split < 8 * (kAcceptThreads / 32)) --split;
    }
    const AcceptArgs a{p, q, draft_tok, u_acc, u_smp, gamma, vocab, q_indptr, ctx_len, acc_len, out_tok, new_ctx_len, status,
                       split, sp.scratch, sp.counters};
    if (split == 1) return launch_kernel(spec_accept_kernel, dim3(batch), dim3(kAcceptThreads), smem, stream, pdl, a);
    return launch_kernel(spec_accept_split_kernel, dim3(batch * split), dim3(kAcceptThreads), smem, stream, pdl, a);
}

}  // namespace nsd
