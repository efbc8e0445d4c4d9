// The part of the epilogue that the two tensor-core kernels (16-bit and TF32x3) share: one epilogue group
// (128 threads, thread <-> output row) works through its 128-column half of a tile whose accumulator sits in
// tensor memory, 32 columns at a time -- bias, activation, scale, then either the store of Y or the row
// statistic of the reduction -- and, for the reductions, leaves its per-row partial in the workspace, where the
// group that arrives last at the row strip folds the parts in part order.  The kernels differ in the accuracy of
// the activations, in how a chunk of Y is stored (packed 16-bit or fp32) and in their barriers, which they pass in.
#pragma once

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace forge {

// What a thread has gathered over its row of the half tile.
struct HalfTileRow {
    float red;              // row sum or maximum (sum / max / mean chain)
    float mx, se, tl;       // (max, sum exp) and the target's logit (log-sum-exp / cross-entropy)
};

// One sweep over the CHUNKS 32-column chunks of the half tile at tensor-memory address `taddr` (columns n0.. of
// the output).  `sb`: the half tile's bias as fp32 in shared memory; `sub`: the vector the mean chain subtracts
// (shared memory; read only for that reduction); `tgt`: this row's class index (cross-entropy) or -1;
// `store(col0, v, nv)`: writes nv values of this thread's row starting at column col0 (called only when there is
// no reduction).
template <bool ACCURATE, int CHUNKS, class Store>
__device__ __forceinline__ void half_tile_sweep(uint32_t taddr, int n0, int N, const Epilogue &e, const float *sb,
                                                const float *sub, int tgt, Store store, HalfTileRow &row)
{
    const bool lse = e.red == FORGE_RED_LOGSUMEXP || e.red == FORGE_RED_CROSS_ENTROPY;
    const bool chain = e.red == FORGE_RED_MEAN_GELU_RESIDUAL;
    const bool fold = e.red == FORGE_RED_SUM || e.red == FORGE_RED_MAX || chain;
    const bool add = e.red != FORGE_RED_MAX;
    row.red = add ? 0.f : -INFINITY;
    row.mx = -INFINITY;
    row.se = row.tl = 0.f;
#pragma unroll 1
    for (int c = 0; c < CHUNKS; ++c) {
        const int col0 = n0 + c * 32;
        if (col0 >= N) break;
        uint32_t r[32];
        ptx::tmem_ld_32x32(taddr + c * 32, r);
        ptx::tmem_ld_wait();
        float v[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]) + sb[c * 32 + j];
        apply_act_array<ACCURATE>(e.act, v, e.scale);
        const int nv = min(32, N - col0);
        if (lse) {
            // online (max, sum exp); the target's logit is picked up on the way; Y is never written
            float cm = -INFINITY;
#pragma unroll
            for (int j = 0; j < 32; ++j) cm = j < nv ? fmaxf(cm, v[j]) : cm;
            const float nm = fmaxf(row.mx, cm);
            float cs = 0.f;
#pragma unroll
            for (int j = 0; j < 32; ++j) cs += j < nv ? lse_exp<ACCURATE>(v[j] - nm) : 0.f;
            row.se = (row.mx == -INFINITY ? 0.f : row.se * lse_exp<ACCURATE>(row.mx - nm)) + cs;
            row.mx = nm;
            if (tgt >= col0 && tgt < col0 + 32) {
#pragma unroll
                for (int j = 0; j < 32; ++j) row.tl = (col0 + j == tgt) ? v[j] : row.tl;
            }
        } else if (fold) {
            if (chain) {
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] -= sub[c * 32 + j];
            }
#pragma unroll
            for (int j = 0; j < 32; ++j)
                if (j < nv) row.red = add ? row.red + v[j] : fmaxf(row.red, v[j]);
        } else {
            store(col0, v, nv);
        }
    }
}

// The reductions: leave this row's partial of part `part` in the workspace, count the group in at the strip's
// counter, and let the group that arrives last fold the strip's `parts` parts in part order: out[row] for sum /
// max / the softmax statistics, gelu(mean) into rowg[row] for the mean chain (whose residual rows the whole grid
// writes once `strips_done` has counted every strip).  `group_sync()` is the group's barrier, `last_flag` a word
// of shared memory of the group, `leader` its thread 0.  One arrival per group by one thread: its release covers
// the group's partials, which the barrier orders before it; its acquire and the next barrier make the other
// groups' partials readable past L1.
template <bool ACCURATE, class GroupSync>
__device__ __forceinline__ void strip_fold(const Epilogue &e, const HalfTileRow &mine, float *partial, int part, int parts, int M, int N,
                                           int row, bool leader, unsigned *counter, int *last_flag, GroupSync group_sync,
                                           float *out, float *rowg, unsigned *strips_done)
{
    const bool lse = e.red == FORGE_RED_LOGSUMEXP || e.red == FORGE_RED_CROSS_ENTROPY;
    const bool chain = e.red == FORGE_RED_MEAN_GELU_RESIDUAL;
    float4 *part4 = reinterpret_cast<float4 *>(partial);
    if (row < M) {
        if (lse) part4[(size_t)part * M + row] = make_float4(mine.mx, mine.se, mine.tl, 0.f);
        else partial[(size_t)part * M + row] = mine.red;
    }
    group_sync();
    if (leader) *last_flag = (arrive_acq_rel(counter) == (unsigned)(parts - 1));
    group_sync();
    if (!*last_flag) return;
    if (row < M) {
        if (lse) {
            out[row] = fold_row_lse<ACCURATE>(part4, parts, M, row);
        } else {
            const float v = e.red != FORGE_RED_MAX ? fold_row_partials<true>(partial, parts, M, row) : fold_row_partials<false>(partial, parts, M, row);
            if (chain) rowg[row] = apply_act<true>(FORGE_ACT_GELU_ERF, v / (float)N);
            else out[row] = v;
        }
    }
    if (leader) *counter = 0u;          // ready for the next run
    if (chain) {
        // the strip's gelu(mean) values are published; the rows are written at the end, by the whole grid
        group_sync();
        if (leader) arrive_acq_rel(strips_done);
    }
}

}  // namespace forge
