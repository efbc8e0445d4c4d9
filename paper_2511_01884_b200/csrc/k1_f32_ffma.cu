// K1: fp32 fused linear.  Register-tiled FFMA GEMM (128x128 CTA tile, 8x8 per thread),
// 128-bit global loads, double-buffered shared memory, epilogue (bias, activation, scale,
// row sum / max / LayerNorm) applied to the accumulators in registers.
//
// Row reductions across the N-tiles of one row strip:
//   sum/max   per-tile partials in a small workspace, folded in tile order by the CTA that
//             arrives last at the strip's counter (deterministic, no float atomics);
//   layernorm persistent CTAs walk the tiles strip by strip, so the N-tiles of a strip are worked on
//             at about the same time; each tile publishes its per-row (n, mean, M2) triples, waits
//             (bounded) until the strip's counter shows all of them, combines them in tile order and
//             normalises the tile it still holds in registers.  CTAs wait on one another: cooperative
//             launch, and a strip may not have more tiles than there are CTAs.
#include <mutex>

#include "common.cuh"
#include "plan.h"

namespace forge {

constexpr int K1_BM = 128, K1_BN = 128, K1_BK = 16, K1_THREADS = 256, K1_PAD = 4;
constexpr int K1_CTAS_PER_SM = 2;            // the kernels are built for two resident CTAs per SM

struct K1Params {
    const float *X, *W, *b, *gamma, *beta;
    float *out;
    int M, N, K;
    Epilogue e;
    float *partial;        // [tiles_n][M]
    unsigned *counters;    // [tiles_m]
    int tiles_n;
    int out_vec4;          // Y rows can be written with 128-bit stores
    int res_vec4;          // mean chain: X and Y rows ([M,K]) can be moved with 128-bit accesses
    int warm_l2;           // small grids: request the CTA's operand panels into L2 before the k loop
    // (Small grids: K is cut into gridDim.z slices, one CTA each; the slice length and the hand-over
    // area follow from the fields above -- see k1_slice_len().)
    int *status;           // LayerNorm: status word of the bounded strip wait
    unsigned *gen;         // LayerNorm: run index of the strip counters (see run_index_begin)
#ifdef FORGE_DEBUG_BOUNDS
    // extents of `partial` and `counters`.  Only in the bounds-checked build: the code generated for the large tile
    // is sensitive to the size of this structure (two more words cost 5 % on a 4096^3 problem).
    long long ws_floats, ws_counters;
#endif
};
#ifdef FORGE_DEBUG_BOUNDS
#define K1_WS_FLOATS(p) ((p).ws_floats)
#define K1_WS_COUNTERS(p) ((p).ws_counters)
#define K1_SET_EXTENTS(p, f, c) ((p).ws_floats = (f), (p).ws_counters = (c))
#else
#define K1_WS_FLOATS(p) 0ll
#define K1_WS_COUNTERS(p) 0ll
#define K1_SET_EXTENTS(p, f, c) ((void)0)
#endif

// Length of a K slice when K is cut into `slices`: a multiple of the small tile's 32-wide k-tile.
__host__ __device__ inline int k1_slice_len(int K, int slices) { return ((K + slices - 1) / slices + 31) / 32 * 32; }

// One CTA-tile slab (128 rows x 16 k, or 64 rows x 32 k) from a K-major matrix into registers: two float4 per
// thread either way.  k_end is the end of this CTA's range of k (K itself unless K is cut into slices).
template <bool VEC, int T>
__device__ __forceinline__ void k1_fetch(const float *__restrict__ base, int rows_total, int K,
                                         int row0, int kt, int tid, float4 (&r)[2], int k_end)
{
    constexpr int KQ = (T == 1 ? 32 : 16) / 4;          // float4 per row of the slab
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const int idx = tid + i * K1_THREADS;
        const int row = row0 + idx / KQ;
        const int k = kt + (idx % KQ) * 4;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (row < rows_total) {
            const float *src = base + (size_t)row * K + k;
            if (VEC) {
                if (k < k_end) v = __ldg(reinterpret_cast<const float4 *>(src));
            } else {
                if (k + 0 < k_end) v.x = __ldg(src + 0);
                if (k + 1 < k_end) v.y = __ldg(src + 1);
                if (k + 2 < k_end) v.z = __ldg(src + 2);
                if (k + 3 < k_end) v.w = __ldg(src + 3);
            }
        }
        r[i] = v;
    }
}

// Registers -> shared memory, transposed to [k][row] so the inner product reads rows of 4.
template <int T>
__device__ __forceinline__ void k1_stash(float (*S)[64 * T + K1_PAD], int tid, const float4 (&r)[2])
{
    constexpr int KQ = (T == 1 ? 32 : 16) / 4;
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const int idx = tid + i * K1_THREADS;
        const int k = (idx % KQ) * 4;
        // rows of the k-groups 8..15 are stored with bit 3 of the row index flipped: the four
        // k-groups a warp writes at once then fall into four different bank octets
        const int row = (idx / KQ) ^ (((k >> 3) & 1) << 3);
        S[k + 0][row] = r[i].x;
        S[k + 1][row] = r[i].y;
        S[k + 2][row] = r[i].z;
        S[k + 3][row] = r[i].w;
    }
}

// Two fp32 fused multiply-adds per instruction (sm_100 packed-pair FMA): the inner product is
// bound by instruction issue, not by the FMA pipe, when it is written with scalar FFMA.
__device__ __forceinline__ void ffma2(unsigned long long &d, unsigned long long a, unsigned long long b)
{
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(d) : "l"(a), "l"(b));
}
__device__ __forceinline__ unsigned long long pack2(float lo, float hi)
{
    unsigned long long r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(unsigned long long v, float &lo, float &hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}

// T = 2: 128x128 CTA tile, 8x8 accumulators per thread.  T = 1: 64x64 tile, 4x4 per thread, for
// problems with too few 128x128 tiles to occupy the SMs (a grid of a handful of CTAs is bound by
// the FMA rate of the few SMs it runs on, not by the GPU's).
// One output tile (for small grids: one K slice of it).  `run` is the run index of the LayerNorm strip counters.
// LayerNorm of rows with more tiles than CTAs computes every tile twice: ln_pass 1 = statistics only (publish, never
// wait), 2 = recompute, wait for the strip, normalise and store; 0 = both in one visit.  Returns false only when a
// bounded wait gave up.
template <bool VEC, int RED, int T>
__device__ __forceinline__ bool k1_tile(const K1Params &p, const int tile_m, const int tile_n, const unsigned run, const int ln_pass = 0)
{
    constexpr int BM = 64 * T, BN = 64 * T, R = 4 * T;       // tile and per-thread extent
    constexpr int BK = T == 1 ? 32 : K1_BK;                  // the small tile takes longer k steps (fewer round trips)
    __shared__ __align__(16) float As[2][BK][BM + K1_PAD];
    __shared__ __align__(16) float Bs[2][BK][BN + K1_PAD];
    __shared__ float s_mean[BM], s_rstd[BM];
    __shared__ int s_last;

    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;
    const int m0 = tile_m * BM, n0 = tile_n * BN;
    const int M = p.M, N = p.N, K = p.K;

    unsigned long long acc2[R][R / 2];   // acc2[i][j] = accumulators (i, 2j) and (i, 2j+1)
#pragma unroll
    for (int i = 0; i < R; ++i)
#pragma unroll
        for (int j = 0; j < R / 2; ++j) acc2[i][j] = 0ull;

    {
        // this CTA's range of k: the whole of K unless a small grid (T == 1) is cut into gridDim.z slices
        const int k_per = T == 1 ? k1_slice_len(K, (int)gridDim.z) : K, k_lo = T == 1 ? (int)blockIdx.z * k_per : 0;
        const int k_hi = min(K, k_lo + k_per);
        if (p.warm_l2) {
            // A small grid walks K with one tile of look-ahead, i.e. it pays the memory latency once
            // per k-tile.  Asking L2 for both operand panels up front puts all of those requests in
            // flight at once; the k loop then runs at L2 latency.
            const int w_len = k_hi - k_lo;
            const int lines_per_row = (w_len * 4 + 127) / 128;
            const int rows_a = min(BM, M - m0), rows_b = min(BN, N - n0);
            for (int i = tid; i < (rows_a + rows_b) * lines_per_row; i += K1_THREADS) {
                const int r = i / lines_per_row, c = i - r * lines_per_row;
                const float *ptr = r < rows_a ? p.X + (size_t)(m0 + r) * K : p.W + (size_t)(n0 + r - rows_a) * K;
                asm volatile("prefetch.global.L2 [%0];" ::"l"(ptr + k_lo + min(c * 32, w_len - 1)));
            }
        }
        float4 ra[2], rb[2];
        k1_fetch<VEC, T>(p.X, M, K, m0, k_lo, tid, ra, k_hi);
        k1_fetch<VEC, T>(p.W, N, K, n0, k_lo, tid, rb, k_hi);
        k1_stash<T>(As[0], tid, ra);
        k1_stash<T>(Bs[0], tid, rb);
        __syncthreads();

        int buf = 0;
        for (int kt = k_lo; kt < k_hi; kt += BK) {
            const bool more = kt + BK < k_hi;
            if (more) {
                k1_fetch<VEC, T>(p.X, M, K, m0, kt + BK, tid, ra, k_hi);
                k1_fetch<VEC, T>(p.W, N, K, n0, kt + BK, tid, rb, k_hi);
            }
#pragma unroll
            for (int k = 0; k < BK; ++k) {
                const int flip = ((k >> 3) & 1) << 3;          // see k1_stash
                float a[R];
                unsigned long long b[R / 2];                    // column pairs as they lie in memory
#pragma unroll
                for (int q = 0; q < T; ++q) {
                    const float4 av = *reinterpret_cast<const float4 *>(&As[buf][k][64 * q + ((ty * 4) ^ flip)]);
                    const ulonglong2 bv = *reinterpret_cast<const ulonglong2 *>(&Bs[buf][k][64 * q + ((tx * 4) ^ flip)]);
                    a[4 * q + 0] = av.x; a[4 * q + 1] = av.y; a[4 * q + 2] = av.z; a[4 * q + 3] = av.w;
                    b[2 * q + 0] = bv.x; b[2 * q + 1] = bv.y;
                }
#pragma unroll
                for (int i = 0; i < R; ++i) {
                    const unsigned long long ai = pack2(a[i], a[i]);
#pragma unroll
                    for (int j = 0; j < R / 2; ++j) ffma2(acc2[i][j], ai, b[j]);
                }
            }
            if (more) {
                k1_stash<T>(As[buf ^ 1], tid, ra);
                k1_stash<T>(Bs[buf ^ 1], tid, rb);
            }
            __syncthreads();
            buf ^= 1;
        }
    }

    float acc[R][R];
#pragma unroll
    for (int i = 0; i < R; ++i)
#pragma unroll
        for (int j = 0; j < R / 2; ++j) unpack2(acc2[i][j], acc[i][2 * j], acc[i][2 * j + 1]);

    if (T == 1 && gridDim.z > 1) {
        // ---- K slices of one tile: raw accumulators to the workspace, summed by the last to arrive ----
        // the hand-over area and its counters lie behind the row partials and the strip counters
        constexpr bool LSE = RED == FORGE_RED_LOGSUMEXP || RED == FORGE_RED_CROSS_ENTROPY;
        const bool row_partials = p.tiles_n > 1 && (RED == FORGE_RED_SUM || RED == FORGE_RED_MAX || RED == FORGE_RED_MEAN_GELU_RESIDUAL || LSE);
        const size_t row_floats = row_partials ? (LSE ? 4 : 1) * (size_t)p.tiles_n * (size_t)M : 0;
        float4 *slice_partial = reinterpret_cast<float4 *>(p.partial + (row_floats + 3) / 4 * 4);
        unsigned *slice_counters = p.counters + (row_partials ? gridDim.y : 0);
        const int k_slices = (int)gridDim.z;
        const int tile = tile_m * (int)gridDim.x + tile_n;
        float4 *mine = slice_partial + (((size_t)tile * k_slices + blockIdx.z) * K1_THREADS + tid) * (R * R / 4);
        // (the same verdict in every thread: the check is on the tile's whole hand-over area and its counter)
        if (!in_bounds(p.status, BOUNDS_PARTIAL, (long long)(reinterpret_cast<float *>(slice_partial) - p.partial) + (long long)tile * k_slices * K1_THREADS * (R * R),
                       (long long)k_slices * K1_THREADS * (R * R), K1_WS_FLOATS(p)) ||
            !in_bounds(p.status, BOUNDS_COUNTER, (long long)(slice_counters - p.counters) + tile, 1, K1_WS_COUNTERS(p)))
            return true;
#pragma unroll
        for (int i = 0; i < R; ++i)
#pragma unroll
            for (int j = 0; j < R / 4; ++j) mine[i * (R / 4) + j] = make_float4(acc[i][4 * j], acc[i][4 * j + 1], acc[i][4 * j + 2], acc[i][4 * j + 3]);
        // one arrival per CTA by one thread: its release covers what the barrier has ordered before it, its acquire
        // (and the next barrier) what the other slices' CTAs had written (read below past L1)
        __syncthreads();
        if (tid == 0) s_last = (arrive_acq_rel(&slice_counters[tile]) == (unsigned)(k_slices - 1));
        __syncthreads();
        if (!s_last) return true;
#pragma unroll
        for (int i = 0; i < R; ++i)
#pragma unroll
            for (int j = 0; j < R; ++j) acc[i][j] = 0.f;
        for (int sl = 0; sl < k_slices; ++sl) {           // slice order, whichever CTA got here last
            const float4 *src = slice_partial + (((size_t)tile * k_slices + sl) * K1_THREADS + tid) * (R * R / 4);
#pragma unroll
            for (int i = 0; i < R; ++i)
#pragma unroll
                for (int j = 0; j < R / 4; ++j) {
                    const float4 o = __ldcg(src + i * (R / 4) + j);
                    acc[i][4 * j] += o.x; acc[i][4 * j + 1] += o.y; acc[i][4 * j + 2] += o.z; acc[i][4 * j + 3] += o.w;
                }
        }
        __syncthreads();                                   // s_last is reused by the row reductions below
        if (tid == 0) slice_counters[tile] = 0u;           // ready for the next run
    }

    // ---- epilogue: bias, activation, scale, in registers --------------------------------
    if (kDebugBounds && RED != FORGE_RED_NONE && (p.tiles_n > 1 || RED == FORGE_RED_LAYERNORM)) {
        // the rows of this tile's partials in the workspace (one float, or one float4, per row) and the strip's
        // counter, checked before either is touched (the same verdict in every thread)
        constexpr bool WIDE = RED == FORGE_RED_LAYERNORM || RED == FORGE_RED_LOGSUMEXP || RED == FORGE_RED_CROSS_ENTROPY;
        const long long first = (long long)tile_n * M + m0, rows = min(BM, M - m0);
        if (!in_bounds(p.status, BOUNDS_PARTIAL, WIDE ? 4 * first : first, WIDE ? 4 * rows : rows, K1_WS_FLOATS(p)) ||
            !in_bounds(p.status, BOUNDS_COUNTER, tile_m, 1, K1_WS_COUNTERS(p)))
            return true;
    }
    int col[R];
    bool cok[R];
    float bias[R];
#pragma unroll
    for (int j = 0; j < R; ++j) {
        col[j] = n0 + tx * 4 + (j & 3) + (j >> 2) * 64;
        cok[j] = col[j] < N;
        bias[j] = (p.e.has_bias && cok[j]) ? __ldg(p.b + col[j]) : 0.f;
    }
#pragma unroll
    for (int i = 0; i < R; ++i)
#pragma unroll
        for (int j = 0; j < R; ++j) acc[i][j] = p.e.scale * apply_act<true>(p.e.act, acc[i][j] + bias[j]);

    if (RED == FORGE_RED_NONE) {
#pragma unroll
        for (int i = 0; i < R; ++i) {
            const int row = m0 + ty * 4 + (i & 3) + (i >> 2) * 64;
            if (row >= M) continue;
            float *dst = p.out + (size_t)row * N;
            if (p.out_vec4) {
#pragma unroll
                for (int q = 0; q < T; ++q)
                    if (cok[4 * q]) *reinterpret_cast<float4 *>(dst + col[4 * q]) = make_float4(acc[i][4 * q], acc[i][4 * q + 1], acc[i][4 * q + 2], acc[i][4 * q + 3]);
            } else {
#pragma unroll
                for (int j = 0; j < R; ++j)
                    if (cok[j]) dst[col[j]] = acc[i][j];
            }
        }
        return true;
    }

    if (RED == FORGE_RED_SUM || RED == FORGE_RED_MAX || RED == FORGE_RED_MEAN_GELU_RESIDUAL) {
        constexpr bool ADD = RED != FORGE_RED_MAX;                       // row sum (also of the mean chain) or row max
        constexpr bool CHAIN = RED == FORGE_RED_MEAN_GELU_RESIDUAL;      // subtract, row mean, GELU, residual add
        float sub[R];
#pragma unroll
        for (int j = 0; j < R; ++j) sub[j] = (CHAIN && p.gamma && cok[j]) ? __ldg(p.gamma + col[j]) : 0.f;
        // thread -> 16 lanes that share the row (shuffles) -> tile partial
#pragma unroll
        for (int i = 0; i < R; ++i) {
            float v = ADD ? 0.f : -INFINITY;
#pragma unroll
            for (int j = 0; j < R; ++j)
                if (cok[j]) v = ADD ? v + (acc[i][j] - sub[j]) : fmaxf(v, acc[i][j]);
#pragma unroll
            for (int s = 8; s >= 1; s >>= 1) {
                const float o = __shfl_xor_sync(0xffffffffu, v, s);
                v = ADD ? v + o : fmaxf(v, o);
            }
            const int rl = ty * 4 + (i & 3) + (i >> 2) * 64;
            const int row = m0 + rl;
            if (tx == 0 && row < M) {
                if (p.tiles_n > 1) p.partial[(size_t)tile_n * M + row] = v;
                else if (CHAIN) s_mean[rl] = apply_act<true>(FORGE_ACT_GELU_ERF, v / (float)N);
                else p.out[row] = v;
            }
        }
        if (p.tiles_n > 1) {
            // the last CTA to arrive at this row strip folds the partials in tile order
            __syncthreads();
            if (tid == 0) s_last = (arrive_acq_rel(&p.counters[tile_m]) == (unsigned)(p.tiles_n - 1));
            __syncthreads();
            if (!s_last) return true;
            if (tid < BM && m0 + tid < M) {
                const int row = m0 + tid;
                const float v = fold_row_partials<ADD>(p.partial, p.tiles_n, M, row);
                if (CHAIN) s_mean[tid] = apply_act<true>(FORGE_ACT_GELU_ERF, v / (float)N);
                else p.out[row] = v;
            }
            if (tid == 0) p.counters[tile_m] = 0u;     // ready for the next run
        }
        if (CHAIN) {
            // residual add: Y[row, :] = X[row, :] + gelu(mean) for the strip's rows, by the whole CTA
            __syncthreads();
            const int rows = min(BM, M - m0);
            if (p.res_vec4) {
                const int k4 = K >> 2;
                for (int e = tid; e < rows * k4; e += K1_THREADS) {
                    const int r = e / k4, c = e - r * k4;
                    float4 x = __ldg(reinterpret_cast<const float4 *>(p.X + (size_t)(m0 + r) * K) + c);
                    const float g = s_mean[r];
                    x.x += g; x.y += g; x.z += g; x.w += g;
                    reinterpret_cast<float4 *>(p.out + (size_t)(m0 + r) * K)[c] = x;
                }
            } else {
                for (int e = tid; e < rows * K; e += K1_THREADS) {
                    const int r = e / K, c = e - r * K;
                    p.out[(size_t)(m0 + r) * K + c] = __ldg(p.X + (size_t)(m0 + r) * K + c) + s_mean[r];
                }
            }
        }
        return true;
    }

    if (RED == FORGE_RED_LOGSUMEXP || RED == FORGE_RED_CROSS_ENTROPY) {
        constexpr bool CE = RED == FORGE_RED_CROSS_ENTROPY;
        const int *target = reinterpret_cast<const int *>(p.gamma);          // class index per row (CE)
        float4 *part4 = reinterpret_cast<float4 *>(p.partial);               // (max, sum exp, target logit, -)
#pragma unroll
        for (int i = 0; i < R; ++i) {
            const int row = m0 + ty * 4 + (i & 3) + (i >> 2) * 64;
            float mx = -INFINITY, se = 0.f, tl = 0.f;
#pragma unroll
            for (int j = 0; j < R; ++j)
                if (cok[j]) mx = fmaxf(mx, acc[i][j]);
#pragma unroll
            for (int j = 0; j < R; ++j)
                if (cok[j]) se += expf(acc[i][j] - mx);
            if (CE && row < M) {
                const int t = __ldg(target + row);
#pragma unroll
                for (int j = 0; j < R; ++j)
                    if (cok[j] && col[j] == t) tl = acc[i][j];
            }
            // the 16 lanes that share the row: shuffles, no block-wide barrier
#pragma unroll
            for (int s = 8; s >= 1; s >>= 1) {
                const float om = __shfl_xor_sync(0xffffffffu, mx, s);
                const float os = __shfl_xor_sync(0xffffffffu, se, s);
                tl += __shfl_xor_sync(0xffffffffu, tl, s);                    // exactly one lane holds it
                lse_merge<true>(mx, se, om, os);
            }
            if (tx == 0 && row < M) {
                if (p.tiles_n == 1) p.out[row] = mx + logf(se) - tl;
                else part4[(size_t)tile_n * M + row] = make_float4(mx, se, tl, 0.f);
            }
        }
        if (p.tiles_n == 1) return true;
        __syncthreads();
        if (tid == 0) s_last = (arrive_acq_rel(&p.counters[tile_m]) == (unsigned)(p.tiles_n - 1));
        __syncthreads();
        if (!s_last) return true;
        if (tid < BM && m0 + tid < M) {
            p.out[m0 + tid] = fold_row_lse<true>(part4, p.tiles_n, M, m0 + tid);
        }
        if (tid == 0) p.counters[tile_m] = 0u;
        return true;
    }

    if (RED == FORGE_RED_LAYERNORM) {
        float4 *stats = reinterpret_cast<float4 *>(p.partial);      // [tiles_n][M] (n, mean, M2, -)
        // per-thread statistics of its <= 8 columns of each row, two sweeps over registers, then the 16 lanes
        // that share the row
#pragma unroll
        for (int i = 0; i < R; ++i) {
            RowStat st;
            float sum = 0.f;
            st.n = 0.f;
#pragma unroll
            for (int j = 0; j < R; ++j)
                if (cok[j]) { sum += acc[i][j]; st.n += 1.f; }
            st.mean = st.n > 0.f ? sum / st.n : 0.f;
            st.m2 = 0.f;
#pragma unroll
            for (int j = 0; j < R; ++j)
                if (cok[j]) { const float d = acc[i][j] - st.mean; st.m2 = fmaf(d, d, st.m2); }
#pragma unroll
            for (int sft = 1; sft <= 8; sft <<= 1) st = merge_stat(st, shfl_xor_stat(st, sft));
            const int row = m0 + ty * 4 + (i & 3) + (i >> 2) * 64;
            if (ln_pass != 2 && tx == 0 && row < M) stats[(size_t)tile_n * M + row] = make_float4(st.n, st.mean, st.m2, 0.f);
        }
        // publish, then wait (bounded) for the strip's other tiles: one arrival per CTA by one thread (release: the
        // CTA's triples, ordered before it by the barrier; the acquiring polls and the next barrier make the other
        // tiles' triples readable past L1)
        __syncthreads();
        if (tid == 0) {
            if (ln_pass != 2) arrive_acq_rel(&p.counters[tile_m]);
            s_last = (ln_pass == 1 || wait_counter<0>(&p.counters[tile_m], run * (unsigned)p.tiles_n, p.status, SITE_ARRIVAL, tile_m)) ? 1 : 0;
        }
        __syncthreads();
        if (!s_last) return false;
        if (ln_pass == 1) return true;
        // the strip's tiles combined in tile order, all at once (same result in every CTA):
        // mean = sum n_i mean_i / sum n_i,  M2 = sum (M2_i + n_i (mean_i - mean)^2)
        if (tid < BM && m0 + tid < M) {
            s_mean[tid] = combine_row_moments<false>(stats, p.tiles_n, M, m0 + tid, p.e.eps, s_rstd[tid]);
        }
        __syncthreads();
        float g[R], be[R];
#pragma unroll
        for (int j = 0; j < R; ++j) {
            g[j] = cok[j] ? __ldg(p.gamma + col[j]) : 0.f;
            be[j] = cok[j] ? __ldg(p.beta + col[j]) : 0.f;
        }
#pragma unroll
        for (int i = 0; i < R; ++i) {
            const int rl = ty * 4 + (i & 3) + (i >> 2) * 64;
            const int row = m0 + rl;
            if (row >= M) continue;
            const float mu = s_mean[rl], rs = s_rstd[rl];
            float *dst = p.out + (size_t)row * N;
            float y[R];
#pragma unroll
            for (int j = 0; j < R; ++j) y[j] = (acc[i][j] - mu) * rs * g[j] + be[j];
            if (p.out_vec4) {
#pragma unroll
                for (int q = 0; q < T; ++q)
                    if (cok[4 * q]) *reinterpret_cast<float4 *>(dst + col[4 * q]) = make_float4(y[4 * q], y[4 * q + 1], y[4 * q + 2], y[4 * q + 3]);
            } else {
#pragma unroll
                for (int j = 0; j < R; ++j)
                    if (cok[j]) dst[col[j]] = y[j];
            }
        }
    }
    return true;
}

// Grid: one CTA per tile (and K slice), blockIdx = (N-tile, M-tile, slice).  LayerNorm: a one-dimensional grid of
// persistent CTAs that take the tiles strip by strip.
template <bool VEC, int RED, int T>
__global__ void __launch_bounds__(K1_THREADS, K1_CTAS_PER_SM) k1_f32_ffma_kernel(const K1Params p)
{
    if (RED == FORGE_RED_LAYERNORM) {
        const unsigned run = run_index_begin(p.gen);
        const int tiles = (int)((p.M + 64 * T - 1) / (64 * T)) * p.tiles_n;
        // a strip with more tiles than the grid has CTAs cannot wait for itself: statistics first (no CTA waits in that
        // pass, so the grid always gets through it), then every tile once more
        const bool two_pass = p.tiles_n > (int)gridDim.x;
        bool fine = true;
        for (int pass = two_pass ? 1 : 0; fine && pass <= (two_pass ? 2 : 0); ++pass)
            for (int t = (int)blockIdx.x; t < tiles; t += (int)gridDim.x) {
                if (!k1_tile<VEC, RED, T>(p, t / p.tiles_n, t % p.tiles_n, run, pass)) { fine = false; break; }
                __syncthreads();          // the tile's shared memory is free for the next one
            }
        if (threadIdx.x == 0) run_index_end(p.gen, run);
    } else {
        k1_tile<VEC, RED, T>(p, (int)blockIdx.y, (int)blockIdx.x, 0u);
    }
}

// ---- host side ---------------------------------------------------------------------------
// Small grids (64x64 tiles, at most half an SM's worth of tiles each): K is cut into up to 8 slices of
// at least 64 k so that more SMs take part; a grid of 16 CTAs otherwise spends its time in the k loop
// of 16 SMs.  Returns the slice count and sets the slice length (a multiple of the 32-wide k-tile).
static int k1_slices(const forge_fused_linear_desc_t &d, int sm_count, int64_t tiles)
{
    int64_t s = sm_count / (tiles > 0 ? tiles : 1);
    if (s > 8) s = 8;
    if (s > d.K / 64) s = d.K / 64;
    if (s < 1) s = 1;
    // the kernel derives the slice length from the slice count: settle on a count that reproduces itself
    for (;;) {
        const int per = k1_slice_len((int)d.K, (int)s);
        const int64_t need = (d.K + per - 1) / per;
        if (need == s) return (int)s;
        s = need;
    }
}

forge_status_t k1_plan(const forge_fused_linear_desc_t &d, int sm_count, forge_plan_info_t *info, WorkspaceLayout *wl)
{
    // 64x64 tiles when 128x128 tiles would leave most SMs idle (LayerNorm keeps the large tile:
    // its cluster spans a row)
    const bool small = d.red != FORGE_RED_LAYERNORM &&
                       ((d.M + K1_BM - 1) / K1_BM) * ((d.N + K1_BN - 1) / K1_BN) * 2 <= sm_count;
    const int bm = small ? K1_BM / 2 : K1_BM, bn = small ? K1_BN / 2 : K1_BN;
    const int64_t tiles_m = (d.M + bm - 1) / bm, tiles_n = (d.N + bn - 1) / bn;
    if (tiles_m > 65535 || tiles_n > 0x7fffffff) return FORGE_ERR_UNSUPPORTED;
    if (d.M > 0x7fffffff || d.N > 0x7fffffff || d.K > 0x7fffffff) return FORGE_ERR_UNSUPPORTED;
    // LayerNorm: persistent CTAs; the tiles of a strip wait for one another (a strip with more tiles than CTAs is
    // served by computing every tile twice)
    const int64_t ln_grid = tiles_m * tiles_n < (int64_t)K1_CTAS_PER_SM * sm_count ? tiles_m * tiles_n : (int64_t)K1_CTAS_PER_SM * sm_count;
    info->kernel = FORGE_KERNEL_F32_FFMA;
    info->tile_m = bm;
    info->tile_n = bn;
    info->tile_k = small ? 32 : K1_BK;
    info->stages = 2;
    info->cluster = 1;
    info->threads = K1_THREADS;
    const int slices = small ? k1_slices(d, sm_count, tiles_m * tiles_n) : 1;
    info->grid = d.red == FORGE_RED_LAYERNORM ? ln_grid : tiles_m * tiles_n * slices;
    info->smem_bytes = 0;
    const bool lse = d.red == FORGE_RED_LOGSUMEXP || d.red == FORGE_RED_CROSS_ENTROPY;      // float4 partials
    const bool partials = (d.red == FORGE_RED_SUM || d.red == FORGE_RED_MAX || d.red == FORGE_RED_MEAN_GELU_RESIDUAL || lse) && tiles_n > 1;
    wl->partial_floats = partials ? (lse ? 4 : 1) * (size_t)tiles_n * (size_t)d.M : 0;
    wl->counters = partials ? (size_t)tiles_m : 0;
    if (d.red == FORGE_RED_LAYERNORM) {       // one (n, mean, M2, -) per row and tile; strip counters, then run index and finished-CTA count
        wl->partial_floats = 4 * (size_t)tiles_n * (size_t)d.M;
        wl->counters = (size_t)tiles_m + 2;
    }
    if (slices > 1) {         // hand-over area of the K slices (64x64 floats per tile and slice) after the row partials
        wl->partial_floats = (wl->partial_floats + 3) / 4 * 4 + (size_t)(tiles_m * tiles_n) * slices * 64 * 64;
        wl->counters += (size_t)(tiles_m * tiles_n);
    }
    return FORGE_OK;
}

// LayerNorm: CTAs wait on one another, so the whole grid must be resident at once.
forge_status_t k1_setup(Handle &h)
{
    if (h.d.red != FORGE_RED_LAYERNORM) return FORGE_OK;
    int coop = 0, a = 0, b = 0;
    if (cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, h.d.device) != cudaSuccess || !coop) return FORGE_ERR_CUDA;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&a, k1_f32_ffma_kernel<true, FORGE_RED_LAYERNORM, 2>, K1_THREADS, 0) != cudaSuccess ||
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b, k1_f32_ffma_kernel<false, FORGE_RED_LAYERNORM, 2>, K1_THREADS, 0) != cudaSuccess)
        return FORGE_ERR_CUDA;
    return (int64_t)(a < b ? a : b) * h.sm_count >= h.info.grid ? FORGE_OK : FORGE_ERR_CUDA;
}

template <bool VEC, int RED, int T = 2>
static forge_status_t k1_launch_t(const K1Params &p, dim3 grid, cudaStream_t stream)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(K1_THREADS);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    if (RED == FORGE_RED_LAYERNORM && cooperative_launch_enabled()) {
        attr[0].id = cudaLaunchAttributeCooperative;
        attr[0].val.cooperative = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
    }
    return cudaLaunchKernelEx(&cfg, k1_f32_ffma_kernel<VEC, RED, T>, p) == cudaSuccess ? FORGE_OK : FORGE_ERR_CUDA;
}

forge_status_t k1_launch(Handle &h, const RunArgs &a)
{
    const forge_fused_linear_desc_t &d = h.d;
    K1Params p;
    p.X = (const float *)a.X;
    p.W = (const float *)a.W;
    p.b = (const float *)a.b;
    p.gamma = (const float *)a.gamma;
    p.beta = (const float *)a.beta;
    p.out = (float *)a.out;
    p.M = (int)d.M;
    p.N = (int)d.N;
    p.K = (int)d.K;
    p.e = Epilogue{(int)d.act, (int)d.red, d.scale, d.ln_eps, d.has_bias};
    p.partial = h.ws.partial;
    p.counters = h.ws.counters;
    p.status = h.ws.status;
    K1_SET_EXTENTS(p, h.ws.partial_floats, h.ws.counter_words);
    const int bm = h.info.tile_m, bn = h.info.tile_n;          // 128 or 64
    p.warm_l2 = (h.info.grid < h.sm_count) && (d.K <= 4096);   // latency-bound grids with modest panels
    p.tiles_n = (int)((d.N + bn - 1) / bn);
    p.out_vec4 = (d.N % 4 == 0) && ((uintptr_t)a.out % 16 == 0);
    p.res_vec4 = (d.K % 4 == 0) && ((uintptr_t)a.out % 16 == 0) && ((uintptr_t)a.X % 16 == 0);
    const int64_t tiles_m = (d.M + bm - 1) / bm;
    const int k_slices = bm != K1_BM ? k1_slices(d, h.sm_count, tiles_m * p.tiles_n) : 1;
    p.gen = h.ws.counters + tiles_m;          // LayerNorm: behind the strip counters
    const dim3 grid = d.red == FORGE_RED_LAYERNORM ? dim3((unsigned)h.info.grid)
                                                   : dim3((unsigned)p.tiles_n, (unsigned)tiles_m, (unsigned)k_slices);
    const bool vec = (d.K % 4 == 0) && ((uintptr_t)a.X % 16 == 0) && ((uintptr_t)a.W % 16 == 0);
#define K1_CASE(R)                                                                                   \
    case R:                                                                                          \
        if (bm == K1_BM)                                                                             \
            return vec ? k1_launch_t<true, R, 2>(p, grid, a.stream) : k1_launch_t<false, R, 2>(p, grid, a.stream); \
        return vec ? k1_launch_t<true, R, 1>(p, grid, a.stream) : k1_launch_t<false, R, 1>(p, grid, a.stream);
    switch (d.red) {
        K1_CASE(FORGE_RED_NONE)
        K1_CASE(FORGE_RED_SUM)
        K1_CASE(FORGE_RED_MAX)
        K1_CASE(FORGE_RED_LAYERNORM)
        K1_CASE(FORGE_RED_MEAN_GELU_RESIDUAL)
        K1_CASE(FORGE_RED_LOGSUMEXP)
        K1_CASE(FORGE_RED_CROSS_ENTROPY)
    }
#undef K1_CASE
    return FORGE_ERR_INVALID_ARG;
}

// ---- row sum / max without any allocation ---------------------------------------------------
// Scratch of forge_fused_linear_f32_reduce_static(): one fixed array per GPU that loads this
// library, held until the process exits.  Layout: arrival counters (one per 128-row strip,
// padded to 256 bytes), then the per-tile row partials [tiles_n][M].
constexpr size_t K1_STATIC_SCRATCH_BYTES = FORGE_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char k1_static_scratch[K1_STATIC_SCRATCH_BYTES];

constexpr int K1_MAX_DEVICES = 64;
static void *k1_static_scratch_addr[K1_MAX_DEVICES];      // device address of the array, per device
static std::mutex k1_static_mutex;

// `k1_static_scratch` names a host-side shadow here; the address the kernel needs comes from
// the runtime, once per device, with that device current.
static forge_status_t k1_static_scratch_on_current_device(void **addr)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= K1_MAX_DEVICES) return FORGE_ERR_CUDA;
    std::lock_guard<std::mutex> lock(k1_static_mutex);
    if (!k1_static_scratch_addr[dev]) {
        int major = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess || major != 10)
            return FORGE_ERR_CUDA;
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, k1_static_scratch) != cudaSuccess || !ptr) {
            cudaGetLastError();
            return FORGE_ERR_CUDA;
        }
        k1_static_scratch_addr[dev] = ptr;
    }
    *addr = k1_static_scratch_addr[dev];
    return FORGE_OK;
}

}  // namespace forge

extern "C" forge_status_t forge_fused_linear_f32_reduce_static(int64_t M, int64_t N, int64_t K, forge_act_t act,
                                                               forge_red_t red, float scale, const void *X,
                                                               const void *W, const void *b, void *out,
                                                               void *cuda_stream)
{
    using namespace forge;
    if (M <= 0 || N <= 0 || K <= 0 || !X || !W || !out) return FORGE_ERR_INVALID_ARG;
    if (act < FORGE_ACT_IDENTITY || act > FORGE_ACT_SILU || !(scale == scale)) return FORGE_ERR_INVALID_ARG;
    if (red != FORGE_RED_SUM && red != FORGE_RED_MAX) return FORGE_ERR_INVALID_ARG;
    if (((uintptr_t)X | (uintptr_t)W | (uintptr_t)b | (uintptr_t)out) % 4 != 0) return FORGE_ERR_INVALID_ARG;
    if (M > 0x7fffffff || N > 0x7fffffff || K > 0x7fffffff) return FORGE_ERR_SCRATCH_LIMIT;
    const int64_t tiles_m = (M + K1_BM - 1) / K1_BM, tiles_n = (N + K1_BN - 1) / K1_BN;
    if (tiles_m > 65535) return FORGE_ERR_SCRATCH_LIMIT;
    const size_t counter_bytes = (((size_t)tiles_m * sizeof(unsigned) + 255) / 256) * 256;
    const size_t partial_bytes = tiles_n > 1 ? (size_t)tiles_n * (size_t)M * sizeof(float) : 0;
    if (counter_bytes + partial_bytes > K1_STATIC_SCRATCH_BYTES) return FORGE_ERR_SCRATCH_LIMIT;

    void *scratch = nullptr;
    const forge_status_t st = k1_static_scratch_on_current_device(&scratch);
    if (st != FORGE_OK) return st;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    // the array keeps whatever the previous call left: the arrival counters must start at zero
    if (cudaMemsetAsync(scratch, 0, counter_bytes, stream) != cudaSuccess) return FORGE_ERR_CUDA;

    K1Params p;
    p.X = (const float *)X;
    p.W = (const float *)W;
    p.b = (const float *)b;
    p.gamma = nullptr;
    p.beta = nullptr;
    p.out = (float *)out;
    p.M = (int)M;
    p.N = (int)N;
    p.K = (int)K;
    p.e = Epilogue{(int)act, (int)red, scale, 0.f, b != nullptr};
    p.counters = (unsigned *)scratch;
    p.partial = (float *)((unsigned char *)scratch + counter_bytes);
    p.tiles_n = (int)tiles_n;
    p.out_vec4 = 0;
    p.res_vec4 = 0;
    p.warm_l2 = 0;
    p.status = nullptr;
    p.gen = nullptr;
    K1_SET_EXTENTS(p, (long long)((K1_STATIC_SCRATCH_BYTES - counter_bytes) / sizeof(float)), (long long)(counter_bytes / sizeof(unsigned)));
    const dim3 grid((unsigned)tiles_n, (unsigned)tiles_m);
    const bool vec = (K % 4 == 0) && ((uintptr_t)X % 16 == 0) && ((uintptr_t)W % 16 == 0);
    if (red == FORGE_RED_SUM)
        return vec ? k1_launch_t<true, FORGE_RED_SUM>(p, grid, stream) : k1_launch_t<false, FORGE_RED_SUM>(p, grid, stream);
    return vec ? k1_launch_t<true, FORGE_RED_MAX>(p, grid, stream) : k1_launch_t<false, FORGE_RED_MAX>(p, grid, stream);
}
