// Speculative acceptance straight from the target's logits: the softmax with temperature
// that turns logits into the p of the acceptance rule (Section 1's cited rule: accept
// while u < min(1, p/q), residual resampling, bonus token) is fused into the kernel, so
// the [batch][gamma+1][vocab] probability tensor is never written or re-read.
//
// One CTA at a time per request; a persistent grid of one CTA (1024 threads) per SM takes the requests from a
// counter.  That bounds the rows in flight to one per SM (~90 MB at the Qwen3 vocabulary), so the draw's second
// read of the rejected row finds it in L2; with a CTA per request and four resident per SM, 512 rows (~310 MB) were
// in flight and that read went to DRAM again.  Rows are swept in order and only as far as needed: row i costs
// one pass (block-wide max and sum of exponentials, kept online per thread and merged
// through shared memory), after which warp 0 can test draft i; the first rejection ends
// the sweep.  The draw then re-reads row n (an L2 hit: one row is ~0.6 MB) together with
// the draft row, forming p on the fly, with the same segment-sum / prefix / finish-inside
// scheme as spec_accept_kernel.  Greedy mode (temperature 0) replaces max/sum by a
// block-wide argmax (smallest index on ties) and needs neither q nor uniforms.
// Exponentials are ex2.approx in fp32 with log2(e)/T folded into the argument; sums and
// compares are fp64.  A decision can therefore differ from an all-fp64 evaluation only
// within fp32 rounding of p at a decision or CDF boundary.
//
// Feed.  Where rows start on 16-byte boundaries and hold whole 16-byte pieces (vocab a multiple of
// 4 for fp32, of 8 for bf16) they do not travel through registers one load at a time: every
// thread copies its own 16-byte pieces of the next tiles with cp.async into a ring of 16 KiB tiles in shared memory and reads them back
// itself, so a CTA keeps up to 176 KiB in flight with no barrier of any kind and no registers
// held.  Each thread sees the same elements in the same order as with direct loads, so the two
// feeds give identical results; other shapes use direct loads.
#include <cuda_bf16.h>

#include <algorithm>

#include "nsd_internal.h"

namespace nsd {
namespace {

constexpr int kThreads = 1024;                  // one CTA per SM (see the kernel): all of an SM's loads come from it
constexpr int kWarps = kThreads / 32;
constexpr int kSeg = 128;                       // tokens per segment of the draw
constexpr int kAhead = 32;                      // drafts per request whose scalars are fetched ahead
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kStatsSlack = 8.0f;             // log2 units a logit may exceed the running reference by

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ float to_float(float v) { return v; }
__device__ __forceinline__ float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }

// Four consecutive logits starting at token k0 (a multiple of 4); tokens past the vocabulary read as -inf.
template <typename T>
__device__ __forceinline__ float4 load4(const T* row, int k0, int vocab, bool vec_ok) {
    float4 z;
    if (vec_ok) {
        if constexpr (sizeof(T) == 4) {
            z = __ldg(reinterpret_cast<const float4*>(row + k0));
        } else {
            const uint2 raw = __ldg(reinterpret_cast<const uint2*>(row + k0));
            const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162*>(&raw.x);
            const __nv_bfloat162 b = *reinterpret_cast<const __nv_bfloat162*>(&raw.y);
            z = make_float4(__low2float(a), __high2float(a), __low2float(b), __high2float(b));
        }
    } else {
        z.x = k0 + 0 < vocab ? to_float(row[k0 + 0]) : -INFINITY;
        z.y = k0 + 1 < vocab ? to_float(row[k0 + 1]) : -INFINITY;
        z.z = k0 + 2 < vocab ? to_float(row[k0 + 2]) : -INFINITY;
        z.w = k0 + 3 < vocab ? to_float(row[k0 + 3]) : -INFINITY;
    }
    return z;
}

struct Shared {
    float red_m[kWarps];
    double red_s[kWarps];
    int red_i[kWarps];
    float row_max;        // M of the current row: a reference within kStatsSlack (log2 units) of its maximum
    double row_sum;       // S = sum_k 2^((z_k - M) * c)
    int row_argmax;
    int n;                // accepted length once decided, else -1
    int found_seg;
    int token;
    double total;
    int dx[kAhead];       // draft tokens, their uniforms and their draft probabilities, fetched ahead of the sweeps
    float du[kAhead];
    float dq[kAhead];
};

// Values one thread takes per iteration of a row sweep: one 16-byte piece (4 fp32 or 8 bf16 values).
template <typename T>
constexpr int kGroup = 16 / (int)sizeof(T);

// Eight bf16 values held in four 32-bit words, as two groups of four floats.
__device__ __forceinline__ void bf16x8_to_float(const uint4 raw, float4& lo, float4& hi) {
    const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162*>(&raw.x), b = *reinterpret_cast<const __nv_bfloat162*>(&raw.y);
    const __nv_bfloat162 c = *reinterpret_cast<const __nv_bfloat162*>(&raw.z), d = *reinterpret_cast<const __nv_bfloat162*>(&raw.w);
    lo = make_float4(__low2float(a), __high2float(a), __low2float(b), __high2float(b));
    hi = make_float4(__low2float(c), __high2float(c), __low2float(d), __high2float(d));
}

// Sweep of one row with direct loads: thread tid takes the groups tid, tid + 512, ... of kGroup<T> consecutive values
// and hands them to add4(four values, index of the first), four at a time in index order.  (The shared-memory ring
// walks the same elements in the same order.)
template <typename T, class Add4>
__device__ __forceinline__ void direct_sweep(const T* row, int vocab, bool vec_ok, Add4 add4) {
    if constexpr (sizeof(T) == 4) {
        const int n4 = (vocab + 3) / 4;
#pragma unroll 4
        for (int k4 = threadIdx.x; k4 < n4; k4 += kThreads) add4(load4(row, k4 * 4, vocab, vec_ok), k4 * 4);
    } else {
        const bool vec16_ok = (vocab % 8 == 0) && (reinterpret_cast<uintptr_t>(row) % 16 == 0);
        const int n8 = (vocab + 7) / 8;
#pragma unroll 2
        for (int k8 = threadIdx.x; k8 < n8; k8 += kThreads) {
            const int k0 = k8 * 8;
            if (vec16_ok) {
                float4 lo, hi;
                bf16x8_to_float(__ldg(reinterpret_cast<const uint4*>(row + k0)), lo, hi);
                add4(lo, k0);
                add4(hi, k0 + 4);
            } else {
                add4(load4(row, k0, vocab, vec_ok), k0);
                if (k0 + 4 < vocab) add4(load4(row, k0 + 4, vocab, vec_ok), k0 + 4);
            }
        }
    }
}

// Online update of one thread's running (reference, sum of exponentials relative to it) with four more logits.
// The reference m is raised only when a logit exceeds it by more than `slack` (= kStatsSlack / c, i.e. when an
// exponential would exceed 2^kStatsSlack): after the first tiles of a row that is rare, whereas an exact running
// maximum changes in some lane of a warp on almost every iteration and makes the whole warp take the rescaling path.
// Any reference gives the same softmax; the sums stay below 2^kStatsSlack * vocab, far inside fp32.
__device__ __forceinline__ void stats_add4(const float4 z, float c, float slack, float& m, float& s) {
    const float zm = fmaxf(fmaxf(z.x, z.y), fmaxf(z.z, z.w));
    if (zm > m + slack) {
        s *= ex2_approx((m - zm) * c);          // m = -inf: s is 0 and stays 0
        m = zm;
    }
    if (m > -INFINITY)
        s += ex2_approx((z.x - m) * c) + ex2_approx((z.y - m) * c) + ex2_approx((z.z - m) * c) + ex2_approx((z.w - m) * c);
}

// Merges the threads' (m, s) pairs into the row's reference (the largest of the threads') and its sum
// (sh.row_max, sh.row_sum).
__device__ void stats_finish(float m, float s, float c, Shared& sh) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    float wm = m;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) wm = fmaxf(wm, __shfl_xor_sync(0xffffffffu, wm, o));
    double ws = (m > -INFINITY) ? (double)s * (double)ex2_approx((m - wm) * c) : 0.0;
    ws = warp_sum(ws);
    if (lane == 0) {
        sh.red_m[warp] = wm;
        sh.red_s[warp] = ws;
    }
    __syncthreads();
    if (warp == 0) {
        const float pm = lane < kWarps ? sh.red_m[lane] : -INFINITY;
        float bm = pm;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, o));
        double bs = (lane < kWarps && pm > -INFINITY) ? sh.red_s[lane] * (double)ex2_approx((pm - bm) * c) : 0.0;
        bs = warp_sum(bs);
        if (lane == 0) {
            sh.row_max = bm;
            sh.row_sum = bs;
        }
    }
    __syncthreads();
}

// Block-wide reference and sum of exponentials of one row, direct loads: every thread keeps a running (m, s) pair.
template <typename T>
__device__ void row_stats(const T* row, int vocab, bool vec_ok, float c, Shared& sh) {
    float m = -INFINITY, s = 0.f;
    const float slack = kStatsSlack / c;
    direct_sweep(row, vocab, vec_ok, [&](const float4 z, int) { stats_add4(z, c, slack, m, s); });
    stats_finish(m, s, c, sh);
}

// Running argmax of one thread: largest value, smallest index among equals, NaN never wins.
__device__ __forceinline__ void argmax_add4(const float4 z, int k0, int vocab, float& bv, int& bi) {
    const float v[4] = {z.x, z.y, z.z, z.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int k = k0 + j;
        if (k < vocab && (v[j] > bv || (bi < 0 && v[j] == v[j]))) {      // strictly greater, or the first non-NaN
            bv = v[j];
            bi = k;
        }
    }
}

// Merges the threads' candidates into the row's argmax (sh.row_argmax).
__device__ void argmax_finish(float bv, int bi, Shared& sh) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    auto better = [](float v1, int i1, float v2, int i2) {   // is (v1, i1) ahead of (v2, i2)?
        if (i1 < 0) return false;
        if (i2 < 0) return true;
        return v1 > v2 || (v1 == v2 && i1 < i2);
    };
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (better(ov, oi, bv, bi)) bv = ov, bi = oi;
    }
    if (lane == 0) {
        sh.red_m[warp] = bv;
        sh.red_i[warp] = bi;
    }
    __syncthreads();
    if (warp == 0) {
        bv = lane < kWarps ? sh.red_m[lane] : -INFINITY;
        bi = lane < kWarps ? sh.red_i[lane] : -1;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
            const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
            if (better(ov, oi, bv, bi)) bv = ov, bi = oi;
        }
        if (lane == 0) sh.row_argmax = bi;
    }
    __syncthreads();
}

// Block-wide argmax of one row, direct loads.
template <typename T>
__device__ void row_argmax(const T* row, int vocab, bool vec_ok, Shared& sh) {
    float bv = -INFINITY;
    int bi = -1;
    direct_sweep(row, vocab, vec_ok, [&](const float4 z, int k0) { argmax_add4(z, k0, vocab, bv, bi); });
    argmax_finish(bv, bi, sh);
}

}  // namespace
}  // namespace nsd

#include "spec_accept_logits_ring.inc"
#include "spec_accept_logits_kernel.inc"
