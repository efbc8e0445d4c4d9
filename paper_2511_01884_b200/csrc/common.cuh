// Shared definitions of the fused linear kernels: epilogue arithmetic, row statistics,
// the device status word.  Everything here is device- or host-inline; no state.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "../../include/forge.h"

namespace forge {

// Element-wise part of the epilogue: bias was already added to z.
struct Epilogue {
    int act;        // forge_act_t
    int red;        // forge_red_t
    float scale;
    float eps;
    int has_bias;
};

// Status word layout: 0 = ok; otherwise (FORGE_ERR_TIMEOUT << 16) | location code.
enum WaitSite : int {
    SITE_TMA_FULL = 1, SITE_STAGE_EMPTY = 2, SITE_ACC_FULL = 3, SITE_ACC_EMPTY = 4,
    SITE_ARRIVAL = 5, SITE_SPLIT = 8
};

// Words 1..3 of the status area describe the first report: a caller-chosen detail word, the
// CTA index and the thread index.
__device__ __forceinline__ void report_status(int *status, int code, int site, int detail)
{
    if (atomicCAS(status, 0, (code << 16) | site) == 0) {
        status[1] = detail;
        status[2] = (int)blockIdx.x;
        status[3] = (int)threadIdx.x;
    }
}
__device__ __forceinline__ void report_timeout(int *status, int site, int detail = 0) { report_status(status, FORGE_ERR_TIMEOUT, site, detail); }

// ---- bounds-checked build ------------------------------------------------------------------------
// With -DFORGE_DEBUG_BOUNDS every offset into the shared-memory ring, every tensor-memory column range and
// every workspace index a kernel computes is compared with the extent of its allocation before it is used;
// the first one outside is recorded in the status word (FORGE_ERR_BOUNDS, which allocation, the index) and the
// access is skipped -- never a trap.  In a normal build in_bounds() is the constant true.
enum BoundsSite : int { BOUNDS_RING = 16, BOUNDS_TMEM = 17, BOUNDS_PARTIAL = 18, BOUNDS_COUNTER = 19, BOUNDS_SMEM = 20 };
#ifdef FORGE_DEBUG_BOUNDS
constexpr bool kDebugBounds = true;
#else
constexpr bool kDebugBounds = false;
#endif
__device__ __forceinline__ bool in_bounds(int *status, int site, long long first, long long count, long long extent)
{
    if (!kDebugBounds) return true;
    if (first >= 0 && count >= 0 && first + count <= extent) return true;
    if (status) report_status(status, FORGE_ERR_BOUNDS, site, (int)first);
    return false;
}

// ---- activations -------------------------------------------------------------------
// ACCURATE = true: libm-grade single precision (the fp32 path must stay within 1e-4 of the
// double-precision chain).  ACCURATE = false: hardware approximations (ex2/tanh/rcp), whose
// ~1e-3 relative error sits far below bf16 output rounding.
template <bool ACCURATE>
__device__ __forceinline__ float apply_act(int act, float z)
{
    switch (act) {
    case FORGE_ACT_RELU:
        return fmaxf(z, 0.0f);
    case FORGE_ACT_GELU_ERF:
        // erff is kept on both paths: there is no hardware erf, and a polynomial of the
        // needed accuracy costs about the same.
        return 0.5f * z * (1.0f + erff(z * 0.70710678118654752f));
    case FORGE_ACT_GELU_TANH: {
        const float u = 0.79788456080286536f * (z + 0.044715f * z * z * z);
        float t;
        if (ACCURATE) {
            t = tanhf(u);
        } else {
            asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(u));
        }
        return 0.5f * z * (1.0f + t);
    }
    case FORGE_ACT_SILU:
        if (ACCURATE) {
            return z / (1.0f + expf(-z));
        } else {
            return __fdividef(z, 1.0f + __expf(-z));
        }
    default:
        return z;
    }
}

// v[i] = scale * act(v[i]) for a register array; the activation is selected once, outside
// the element loop.
template <bool ACCURATE, int ACT, int N>
__device__ __forceinline__ void apply_act_fixed(float (&v)[N], float scale)
{
#pragma unroll
    for (int i = 0; i < N; ++i) v[i] = scale * apply_act<ACCURATE>(ACT, v[i]);
}
template <bool ACCURATE, int N>
__device__ __forceinline__ void apply_act_array(int act, float (&v)[N], float scale)
{
    switch (act) {
    case FORGE_ACT_RELU: apply_act_fixed<ACCURATE, FORGE_ACT_RELU>(v, scale); break;
    case FORGE_ACT_GELU_ERF: apply_act_fixed<ACCURATE, FORGE_ACT_GELU_ERF>(v, scale); break;
    case FORGE_ACT_GELU_TANH: apply_act_fixed<ACCURATE, FORGE_ACT_GELU_TANH>(v, scale); break;
    case FORGE_ACT_SILU: apply_act_fixed<ACCURATE, FORGE_ACT_SILU>(v, scale); break;
    default: apply_act_fixed<ACCURATE, FORGE_ACT_IDENTITY>(v, scale); break;
    }
}

// ---- row statistics (count, mean, sum of squared deviations) -------------------------
// Merging rule of Chan, Golub & LeVeque for partitioned samples; the single-pass form of
// the variance that lets LayerNorm statistics be combined across threads, warps and CTAs
// without a second sweep over the data in memory.
struct RowStat {
    float n, mean, m2;
};

__device__ __forceinline__ RowStat merge_stat(RowStat a, RowStat b)
{
    if (b.n == 0.0f) return a;
    if (a.n == 0.0f) return b;
    RowStat r;
    r.n = a.n + b.n;
    const float d = b.mean - a.mean;
    const float f = b.n / r.n;
    r.mean = a.mean + d * f;
    r.m2 = a.m2 + b.m2 + d * d * a.n * f;
    return r;
}

__device__ __forceinline__ RowStat shfl_xor_stat(RowStat s, int mask)
{
    RowStat o;
    o.n = __shfl_xor_sync(0xffffffffu, s.n, mask);
    o.mean = __shfl_xor_sync(0xffffffffu, s.mean, mask);
    o.m2 = __shfl_xor_sync(0xffffffffu, s.m2, mask);
    return o;
}

// ---- log-sum-exp partials ---------------------------------------------------------------
// A set of logits is summarised by (m, s) with m its maximum and s = sum exp(x - m); two
// summaries combine to (max(m1, m2), s1 exp(m1 - m) + s2 exp(m2 - m)).  An empty set is
// (-inf, 0) and must not contribute exp(-inf + inf).
template <bool ACCURATE>
__device__ __forceinline__ float lse_exp(float x) { return ACCURATE ? expf(x) : __expf(x); }

template <bool ACCURATE>
__device__ __forceinline__ void lse_merge(float &m, float &s, float om, float os)
{
    const float nm = fmaxf(m, om);
    const float a = (m == -INFINITY) ? 0.f : s * lse_exp<ACCURATE>(m - nm);
    const float b = (om == -INFINITY) ? 0.f : os * lse_exp<ACCURATE>(om - nm);
    m = nm;
    s = a + b;
}

// ---- counters that CTAs of one launch wait on --------------------------------------------------
__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned *p)
{
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Count an arrival.  Release: everything this thread has observed -- its own writes and, through a
// CTA barrier it has passed, the writes of the CTA's other threads -- is visible to whoever acquires
// the counter later.  Acquire: what earlier arrivals had released is visible to this thread and, after
// another CTA barrier, to the rest of the CTA (which must read it past L1, e.g. with __ldcg).
__device__ __forceinline__ unsigned arrive_acq_rel(unsigned *counter)
{
    unsigned old;
    asm volatile("atom.add.acq_rel.gpu.global.u32 %0, [%1], 1;" : "=r"(old) : "l"(counter) : "memory");
    return old;
}

__device__ __forceinline__ uint64_t wait_clock_ns()
{
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Budget of every device-side wait: about two seconds of wall clock.
constexpr uint64_t kWaitBudgetNs = 2000000000ull;

// Poll until *counter has reached `target` (counters only ever grow; the difference is taken
// modulo 2^32).  Gives up -- returning false -- when another thread has already recorded a give-up
// in the status word or when the budget is spent, in which case the give-up is recorded with
// `site` and `detail`.  SLEEP_NS > 0 backs off between polls.
template <int SLEEP_NS>
__device__ __forceinline__ bool wait_counter(const unsigned *counter, unsigned target, int *status, int site, int detail)
{
    uint64_t t0 = 0;
    for (uint32_t it = 1; (int)(ld_acquire_u32(counter) - target) < 0; ++it) {
        if (SLEEP_NS > 0) __nanosleep(SLEEP_NS);
        if ((it & 0x3f) == 0) {
            if (*(volatile int *)status != 0) return false;
            const uint64_t now = wait_clock_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > kWaitBudgetNs) {
                report_timeout(status, site, detail);
                return false;
            }
        }
    }
    return true;
}

// Run index of a launch whose CTAs wait on one another's arrival counters.  Those counters are
// never reset: every run adds a fixed number of arrivals to each, so run r is complete at r times
// that number.  r itself lives in device memory -- gen[0] = runs completed, gen[1] = CTAs of the
// current run that have finished -- so that nothing about a launch depends on how many launches
// the host has issued before (a launch that failed, or one replayed from a captured graph, sees
// the right index).  Every CTA reads the index when it starts and reports when it ends; the CTA
// that ends last publishes the new count.  One run per handle in flight.
__device__ __forceinline__ unsigned run_index_begin(const unsigned *gen) { return ld_acquire_u32(gen) + 1u; }
__device__ __forceinline__ void run_index_end(unsigned *gen, unsigned run)
{
    if (arrive_acq_rel(gen + 1) == gridDim.x - 1) {      // the next reader is a later launch: nothing else to order
        gen[1] = 0u;
        gen[0] = run;
    }
}

// ---- folds of what the tiles of a row strip leave in the workspace -------------------------------
// All of them walk the parts in part order whichever CTA does the walking, so the result does not depend
// on arrival order; loads are issued eight at a time (a dependent round trip per part made the fold of a
// wide row the longest thing in the kernel) and read past L1 (the values come from other SMs).

// Row sums or maxima: partial[part * M + row], part = 0 .. parts-1.
template <bool ADD>
__device__ __forceinline__ float fold_row_partials(const float *partial, int parts, int M, int row)
{
    float v = __ldcg(&partial[row]);
    int i = 1;
    for (; i + 8 <= parts; i += 8) {
        float o[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) o[u] = __ldcg(&partial[(size_t)(i + u) * M + row]);
#pragma unroll
        for (int u = 0; u < 8; ++u) v = ADD ? v + o[u] : fmaxf(v, o[u]);
    }
    for (; i < parts; ++i) {
        const float o = __ldcg(&partial[(size_t)i * M + row]);
        v = ADD ? v + o : fmaxf(v, o);
    }
    return v;
}

// Softmax statistics (max, sum exp, target logit, -) per part: returns logsumexp - target logit.
template <bool ACCURATE>
__device__ __forceinline__ float fold_row_lse(const float4 *part4, int parts, int M, int row)
{
    float4 f = __ldcg(&part4[row]);
    float mx = f.x, se = f.y, tl = f.z;
    int i = 1;
    for (; i + 8 <= parts; i += 8) {
        float4 g[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) g[u] = __ldcg(&part4[(size_t)(i + u) * M + row]);
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            lse_merge<ACCURATE>(mx, se, g[u].x, g[u].y);
            tl += g[u].z;
        }
    }
    for (; i < parts; ++i) {
        f = __ldcg(&part4[(size_t)i * M + row]);
        lse_merge<ACCURATE>(mx, se, f.x, f.y);
        tl += f.z;
    }
    return mx + (ACCURATE ? logf(se) : __logf(se)) - tl;
}

// LayerNorm: the strip's (n, mean, M2, -) triples combined in one walk, with one division for the mean and
// one for the variance (the pairwise merge costs a division per part).  With d_i = mean_i - mean_0:
//     mean = mean_0 + sum n_i d_i / n,   M2 = sum M2_i + sum n_i d_i^2 - (sum n_i d_i)^2 / n,   n = sum n_i.
// Shifting by the first part's mean keeps the subtraction in M2 harmless: what cancels is of the size of the
// spread of the parts' means, not of the mean itself.  Returns the mean and writes 1 / sqrt(M2 / n + eps).
template <bool ACCURATE>
__device__ __forceinline__ float combine_row_moments(const float4 *stats, int parts, int M, int row, float eps, float &rstd)
{
    const float4 first = __ldcg(&stats[row]);
    float cnt = first.x, s1 = 0.f, s2 = 0.f, m2 = first.z;
    int i = 1;
    for (; i + 8 <= parts; i += 8) {
        float4 o[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) o[u] = __ldcg(&stats[(size_t)(i + u) * M + row]);
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const float d = o[u].y - first.y, nd = o[u].x * d;
            cnt += o[u].x;
            s1 += nd;
            s2 = fmaf(nd, d, s2);
            m2 += o[u].z;
        }
    }
    for (; i < parts; ++i) {
        const float4 o = __ldcg(&stats[(size_t)i * M + row]);
        const float d = o.y - first.y, nd = o.x * d;
        cnt += o.x;
        s1 += nd;
        s2 = fmaf(nd, d, s2);
        m2 += o.z;
    }
    const float inv = 1.0f / cnt, shift = s1 * inv;
    const float var = fmaxf((m2 + s2 - s1 * shift) * inv, 0.f);
    rstd = ACCURATE ? 1.0f / sqrtf(var + eps) : rsqrtf(var + eps);
    return first.y + shift;
}

// (n, mean, M2) of the first nv of 32 values held in registers: two sweeps, no division per element.
__device__ __forceinline__ RowStat chunk_moments(const float (&v)[32], int nv)
{
    RowStat cs;
    cs.n = (float)nv;
    cs.m2 = 0.f;
    if (nv == 32) {
        float sum = 0.f;
#pragma unroll
        for (int j = 0; j < 32; ++j) sum += v[j];
        cs.mean = sum * (1.0f / 32.0f);
#pragma unroll
        for (int j = 0; j < 32; ++j) { const float dlt = v[j] - cs.mean; cs.m2 = fmaf(dlt, dlt, cs.m2); }
    } else {
        float sum = 0.f;
#pragma unroll
        for (int j = 0; j < 32; ++j) sum += j < nv ? v[j] : 0.f;
        cs.mean = sum / cs.n;
#pragma unroll
        for (int j = 0; j < 32; ++j) {
            const float dlt = j < nv ? v[j] - cs.mean : 0.f;
            cs.m2 = fmaf(dlt, dlt, cs.m2);
        }
    }
    return cs;
}

constexpr int ceil_div(int a, int b) { return (a + b - 1) / b; }

// ---- residual rows of the mean chain --------------------------------------------------------------------
// Y[r, :] = X[r, :] + g(r) over `total` 16-byte pieces (`per_row` of them to a row), this thread taking the pieces
// first, first + step, ...  BATCH loads are issued before the first is used: with one load in flight per thread the
// grid keeps well under a megabyte in flight, a fraction of what the memory system needs to stream.  g(row) yields
// the row's addend, add(piece, addend) applies it to the values packed in the piece.  Y is written once and not read
// again here: streaming stores.
template <int BATCH, class Vec, class RowValue, class Add>
__device__ __forceinline__ void residual_rows(const Vec *__restrict__ X, Vec *__restrict__ Y, size_t per_row, size_t total,
                                              size_t first, size_t step, RowValue g, Add add)
{
    static_assert(sizeof(Vec) == 16, "16-byte pieces");
    const bool narrow = total <= 0xffffffffull;              // 32-bit division where the indices allow it
    for (size_t e0 = first; e0 < total; e0 += BATCH * step) {
        Vec x[BATCH];
#pragma unroll
        for (int u = 0; u < BATCH; ++u) {
            const size_t e = e0 + (size_t)u * step;
            if (e < total) x[u] = __ldg(X + e);
        }
#pragma unroll
        for (int u = 0; u < BATCH; ++u) {
            const size_t e = e0 + (size_t)u * step;
            if (e < total) {
                const size_t row = narrow ? (size_t)((uint32_t)e / (uint32_t)per_row) : e / per_row;
                add(x[u], g(row));
                __stcs(Y + e, x[u]);
            }
        }
    }
}

}  // namespace forge
