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
    SITE_ARRIVAL = 5, SITE_STORE = 6, SITE_CLUSTER = 7, SITE_SPLIT = 8
};

// Words 1..3 of the status area describe the first give-up: a caller-chosen detail word, the
// CTA index and the thread index.
__device__ __forceinline__ void report_timeout(int *status, int site, int detail = 0)
{
    if (atomicCAS(status, 0, (int(FORGE_ERR_TIMEOUT) << 16) | site) == 0) {
        status[1] = detail;
        status[2] = (int)blockIdx.x;
        status[3] = (int)threadIdx.x;
    }
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

// Order-preserving map float -> unsigned (for an order-independent atomic max).
__device__ __forceinline__ unsigned float_to_ordered(float f)
{
    const unsigned u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float ordered_to_float(unsigned u)
{
    return __uint_as_float((u & 0x80000000u) ? (u & 0x7fffffffu) : ~u);
}

constexpr int ceil_div(int a, int b) { return (a + b - 1) / b; }

}  // namespace forge
