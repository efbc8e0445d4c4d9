// K3: 16-bit fused linear for a few rows of X (M <= 128), with the operands swapped (HBM-bound: the weight
// matrix is read once and that is the whole cost).
//
// The tensor core computes Z^T = W X^T: up to 128 rows of W are the M dimension of a tcgen05 MMA
// and the (padded) rows of X its N dimension, so a TMA box of W is an operand as it lands -- no
// warp touches the stream.  Each CTA owns a contiguous range of 8-row groups of W sized so that all
// CTAs stream the same number of bytes, and walks it in strips of at most 128 rows.  Warp 0 streams W
// and the matching slice of X (which stays L2-resident) through a ring whose stages hold one to eight
// 64-k boxes; one thread of warp 1 issues four MMAs per box (M = 128, N = padded rows of X, K = 16) into one of two
// tensor-memory accumulators; warps 2..5 read a finished accumulator (thread <-> row of W = output
// column), add the bias, apply the activation and either store Y or reduce over the strip's columns
// with shuffles, then across strips and -- by the CTA that arrives last, in CTA order -- across CTAs.
//
// The MMA always spans 128 rows of shared memory.  Where the strip has fewer rows, the rest of the
// operand is whatever follows the box inside the stage (the X tile, stale bytes); the accumulator rows
// they produce are never read.
//
// Every thread of the CTA stays resident until the common exit barrier, so that no copy can still be
// in flight towards the shared memory of a CTA that has left, and tensor memory is freed after it.
#include "common.cuh"
#include "plan.h"
#include "sm100_ptx.cuh"

namespace forge {

constexpr int K3_BK = 64;                      // k per TMA box: one 128-byte swizzle row
// Boxes per stage (planned per problem, or forced by a tuning build with -DFORGE_K3_KB=1..8).
#ifndef FORGE_K3_KB
#define FORGE_K3_KB 0
#endif
constexpr int K3_MAX_KB = 8;
static_assert(FORGE_K3_KB >= 0 && FORGE_K3_KB <= K3_MAX_KB, "boxes per stage");
constexpr int K3_MAX_ROWS_W = 128;             // rows of W per strip (the MMA's M)
constexpr int K3_MAX_M = 128;                  // rows of X (the MMA's N, padded to a multiple of 16)
constexpr int K3_MAX_STAGES = 16;
constexpr int K3_EPI_WARP0 = 2, K3_EPI_WARPS = 4, K3_EPI_THREADS = K3_EPI_WARPS * 32;
constexpr int K3_THREADS = (K3_EPI_WARP0 + K3_EPI_WARPS) * 32;
constexpr uint32_t K3_A_SPAN = K3_MAX_ROWS_W * K3_BK * 2;     // 16 KiB: what one MMA reads as its first operand

struct K3Smem {
    uint64_t full[K3_MAX_STAGES];
    uint64_t empty[K3_MAX_STAGES];
    uint64_t acc_full[2];
    uint64_t acc_empty[2];
    float red[K3_EPI_WARPS][K3_MAX_M];        // per warp and row of X: sum or max over the warp's 32 columns ...
    float red_s[K3_EPI_WARPS][K3_MAX_M];      // ... softmax: sum of exponentials ...
    float red_t[K3_EPI_WARPS][K3_MAX_M];      // ... and the target's logit
    float fold[4][K3_EPI_THREADS];             // the last CTA's fold: (row, chunk of CTAs) results
    uint32_t tmem_base;
    int last_flag;
    int abort_flag;
};
constexpr size_t K3_SMEM_LIMIT = 232448;       // opt-in shared memory per CTA on this architecture
constexpr size_t K3_RING_BUDGET = (K3_SMEM_LIMIT - 1024 - sizeof(K3Smem)) / 1024 * 1024;

struct K3Params {
    int f16;              // IEEE half (1) or bfloat16 (0) storage
    const uint16_t *b;
    const int *target;    // cross-entropy: class index per row
    void *out;
    int M, N, K;
    Epilogue e;
    float *partial;       // [grid][xr] floats, or float4 (softmax statistics)
    unsigned *counters;   // [1]
    int *status;
    int num_kb;
    int groups;           // N / 8
    int box_groups;       // groups per strip = rows of the W box / 8
    int xr;               // rows of X padded to a multiple of 16
    int stages;
    int kb;               // boxes per stage
    uint32_t stage_bytes; // kb W boxes, then kb X boxes; the last W box is followed by at least 16 KiB - its size
    uint32_t ring_bytes;
    uint32_t tmem_cols;   // power of two >= 2 * xr
    long long ws_floats;  // extent of `partial` (bounds-checked build)
};

__device__ __forceinline__ void k3_epi_sync() { asm volatile("bar.sync 1, %0;" ::"n"(K3_EPI_THREADS) : "memory"); }

// Reduce 16 per-lane values over the 32 lanes of a warp with 16 shuffles instead of 80: at each of the first four
// steps a lane keeps the half of its values that its lane bit selects, sends the other half to the partner lane and
// combines what it receives, so that after them a lane holds one value (index = lane bits 4..1) reduced over 16
// lanes, and one last exchange completes it.  The order of the combinations is fixed.  MODE 0: sums of a; 1: maxima
// of a; 2: softmax statistics (a = max, b = sum of exponentials about it) and sums of c.
template <int MODE, int N>
__device__ __forceinline__ void k3_halve(const float (&a)[2 * N], const float (&b)[2 * N], const float (&c)[2 * N],
                                          float (&ra)[N], float (&rb)[N], float (&rc)[N], bool upper, int sh)
{
#pragma unroll
    for (int i = 0; i < N; ++i) {
        const float keep = upper ? a[N + i] : a[i], send = upper ? a[i] : a[N + i];
        const float got = __shfl_xor_sync(0xffffffffu, send, sh);
        if (MODE == 0) ra[i] = keep + got;
        else if (MODE == 1) ra[i] = fmaxf(keep, got);
        else {
            const float keep_b = upper ? b[N + i] : b[i], send_b = upper ? b[i] : b[N + i];
            const float keep_c = upper ? c[N + i] : c[i], send_c = upper ? c[i] : c[N + i];
            ra[i] = keep; rb[i] = keep_b;
            lse_merge<false>(ra[i], rb[i], got, __shfl_xor_sync(0xffffffffu, send_b, sh));
            rc[i] = keep_c + __shfl_xor_sync(0xffffffffu, send_c, sh);
        }
    }
}
template <int MODE>
__device__ __forceinline__ int k3_reduce16(const float (&a)[16], const float (&b)[16], const float (&c)[16], int lane,
                                            float &oa, float &ob, float &oc)
{
    float a8[8], b8[8], c8[8], a4[4], b4[4], c4[4], a2[2], b2[2], c2[2], a1[1], b1[1], c1[1];
    k3_halve<MODE, 8>(a, b, c, a8, b8, c8, (lane & 16) != 0, 16);
    k3_halve<MODE, 4>(a8, b8, c8, a4, b4, c4, (lane & 8) != 0, 8);
    k3_halve<MODE, 2>(a4, b4, c4, a2, b2, c2, (lane & 4) != 0, 4);
    k3_halve<MODE, 1>(a2, b2, c2, a1, b1, c1, (lane & 2) != 0, 2);
    oa = a1[0]; ob = b1[0]; oc = c1[0];
    const float pa = __shfl_xor_sync(0xffffffffu, oa, 1);
    if (MODE == 0) oa += pa;
    else if (MODE == 1) oa = fmaxf(oa, pa);
    else {
        lse_merge<false>(oa, ob, pa, __shfl_xor_sync(0xffffffffu, ob, 1));
        oc += __shfl_xor_sync(0xffffffffu, oc, 1);
    }
    return (lane >> 1) & 15;
}

__global__ void __launch_bounds__(K3_THREADS, 1)
k3_bf16_skinny_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW, const K3Params p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *ring = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    K3Smem &s = *reinterpret_cast<K3Smem *>(ring + p.ring_bytes);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // this CTA's share of the 8-row groups of W, and its strips
    const int g_lo = (int)((long long)p.groups * blockIdx.x / gridDim.x);
    const int g_hi = (int)((long long)p.groups * (blockIdx.x + 1) / gridDim.x);
    const int strips = (g_hi - g_lo + p.box_groups - 1) / p.box_groups;
    const uint32_t wbox_bytes = (uint32_t)p.box_groups * 8 * K3_BK * 2;       // multiple of 1024
    const uint32_t xbox_bytes = (uint32_t)p.xr * K3_BK * 2;
    const int STAGES = p.stages;

    if (threadIdx.x == 0) {
        for (int i = 0; i < K3_MAX_STAGES; ++i) { ptx::mbar_init(&s.full[i], 1); ptx::mbar_init(&s.empty[i], 1); }
        for (int i = 0; i < 2; ++i) { ptx::mbar_init(&s.acc_full[i], 1); ptx::mbar_init(&s.acc_empty[i], K3_EPI_WARPS); }
        s.abort_flag = 0;
        s.last_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tmap(&tmX);
        ptx::prefetch_tmap(&tmW);
    }
    if (warp == 1) {
        ptx::tmem_alloc(&s.tmem_base, p.tmem_cols);
        ptx::tmem_relinquish();
    }
    // This kernel is short (tens of microseconds), so the gap between two launches matters: let the next launch set
    // itself up on each SM as soon as this CTA leaves it, and touch global memory only once everything earlier in the
    // stream has completed.
    ptx::pdl_launch_dependents();
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = s.tmem_base;
    ptx::pdl_wait();

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (ptx::elect_one()) {
            int slot = 0;
            uint32_t phase = 0;
            bool ok = true;
            // CTAs start at different k: if all of them walked K in lock step, the requests in flight would share their
            // low address bits and pile onto a few DRAM channels
            const int kb_rot = (int)((long long)p.num_kb * blockIdx.x / gridDim.x);
            for (int st = 0; st < strips && ok; ++st) {
                const int row0 = (g_lo + st * p.box_groups) * 8;
                for (int i = 0; i < p.num_kb; ++i) {
                    int kb = i + kb_rot;
                    if (kb >= p.num_kb) kb -= p.num_kb;
                    if (!ptx::mbar_wait(&s.empty[slot], phase ^ 1, p.status, SITE_STAGE_EMPTY, (slot << 16) | (kb & 0xffff))) { ok = false; break; }
                    if (!in_bounds(p.status, BOUNDS_RING, (long long)slot * p.stage_bytes, p.stage_bytes, (long long)p.ring_bytes)) { ok = false; break; }
                    uint8_t *dst = ring + (size_t)slot * p.stage_bytes;
                    ptx::mbar_expect_tx(&s.full[slot], p.kb * (wbox_bytes + xbox_bytes));
                    // a box that starts at or past K, N or M is zero fill and counts in full
                    for (int j = 0; j < p.kb; ++j) {
                        ptx::tma_load_2d(dst + j * wbox_bytes, &tmW, &s.full[slot], (kb * p.kb + j) * K3_BK, row0);
                        ptx::tma_load_2d(dst + p.kb * wbox_bytes + j * xbox_bytes, &tmX, &s.full[slot], (kb * p.kb + j) * K3_BK, 0);
                    }
                    if (++slot == STAGES) { slot = 0; phase ^= 1; }
                }
            }
            if (!ok) s.abort_flag = 1;
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (ptx::elect_one()) {
            const uint32_t idesc = ptx::idesc_16_f32(K3_MAX_ROWS_W, p.xr, p.f16);
            int slot = 0, acc = 0;
            uint32_t phase = 0, acc_phase = 0;
            bool ok = true;
            for (int st = 0; st < strips && ok; ++st) {
                if (!ptx::mbar_wait(&s.acc_empty[acc], acc_phase ^ 1, p.status, SITE_ACC_EMPTY, st)) { ok = false; break; }
                ptx::tc_fence_after();
                if (!in_bounds(p.status, BOUNDS_TMEM, acc * p.xr, p.xr, p.tmem_cols)) { ok = false; break; }
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * p.xr);
                for (int i = 0; i < p.num_kb; ++i) {
                    if (!ptx::mbar_wait(&s.full[slot], phase, p.status, SITE_TMA_FULL, (slot << 16) | (i & 0xffff))) { ok = false; break; }
                    // the first operand spans 16 KiB from the start of each W box
                    if (!in_bounds(p.status, BOUNDS_RING, (long long)slot * p.stage_bytes + (p.kb - 1) * wbox_bytes, K3_A_SPAN, (long long)p.ring_bytes)) { ok = false; break; }
                    ptx::tc_fence_after();
                    const uint8_t *a = ring + (size_t)slot * p.stage_bytes;
                    for (int j = 0; j < p.kb; ++j) {
                        const uint64_t adesc = ptx::smem_desc_k_sw128(a + j * wbox_bytes);
                        const uint64_t bdesc = ptx::smem_desc_k_sw128(a + p.kb * wbox_bytes + j * xbox_bytes);
#pragma unroll
                        for (int k = 0; k < K3_BK / 16; ++k)      // 16 elements = 32 bytes = 2 descriptor units
                            ptx::umma_bf16(d_tmem, adesc + 2 * k, bdesc + 2 * k, idesc, (i != 0) | (j != 0) | (k != 0));
                    }
                    ptx::umma_commit(&s.empty[slot]);
                    if (++slot == STAGES) { slot = 0; phase ^= 1; }
                }
                if (!ok) break;
                ptx::umma_commit(&s.acc_full[acc]);
                if ((acc ^= 1) == 0) acc_phase ^= 1;
            }
            if (!ok) s.abort_flag = 1;
        }
    } else {
        // ---------------- epilogue: thread <-> row of W (output column), 16 rows of X at a time ----------------
        const int q = warp & 3;                              // the quarter of the tensor-memory lanes this warp may read
        const int nl = q * 32 + lane;                        // row of W inside the strip
        const int et = (int)threadIdx.x - 32 * K3_EPI_WARP0;      // 0..127; thread et carries row et of X across strips
        const bool sum = p.e.red == FORGE_RED_SUM;
        const bool reduce = sum || p.e.red == FORGE_RED_MAX;
        const bool softmax = p.e.red == FORGE_RED_LOGSUMEXP || p.e.red == FORGE_RED_CROSS_ENTROPY;
        const float neutral = sum ? 0.f : -INFINITY;
        float running = neutral, running_s = 0.f, running_t = 0.f;
        int acc = 0;
        uint32_t acc_phase = 0;
        bool ok = true;

        for (int st = 0; st < strips; ++st) {
            const int gbase = g_lo + st * p.box_groups;
            const int ng = min(p.box_groups, p.groups - gbase);       // groups present in this strip's box
            const int g = nl >> 3;
            const bool live = g < ng && gbase + g < g_hi;             // in the box, in this CTA's share (hence below N)
            const int n = gbase * 8 + nl;
            const float bias = (live && p.e.has_bias) ? ptx::load16(p.b, (size_t)n, p.f16) : 0.f;
            if (ok && !ptx::mbar_wait(&s.acc_full[acc], acc_phase, p.status, SITE_ACC_FULL, st)) ok = false;
            ptx::tc_fence_after();
            if (ok && !in_bounds(p.status, BOUNDS_TMEM, acc * p.xr, p.xr, p.tmem_cols)) ok = false;
            ok = __all_sync(0xffffffffu, ok);                         // the tensor-memory loads are warp-wide
            if (ok) {
                const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * p.xr);
                for (int c = 0; c < p.xr / 16; ++c) {
                    uint32_t r[16];
                    ptx::tmem_ld_32x16(t_row + (uint32_t)(c * 16), r);
                    ptx::tmem_ld_wait();
                    float v[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]) + bias;
                    apply_act_array<false>(p.e.act, v, p.e.scale);
                    if (reduce) {
                        float x[16], oa, ob, oc;
#pragma unroll
                        for (int i = 0; i < 16; ++i) x[i] = live ? v[i] : neutral;
                        const int idx = sum ? k3_reduce16<0>(x, x, x, lane, oa, ob, oc) : k3_reduce16<1>(x, x, x, lane, oa, ob, oc);
                        if ((lane & 1) == 0) s.red[q][c * 16 + idx] = oa;
                    } else if (softmax) {
                        float mx[16], se[16], tl[16], oa, ob, oc;
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            const int m = c * 16 + i;
                            mx[i] = live ? v[i] : -INFINITY;
                            se[i] = live ? 1.f : 0.f;
                            tl[i] = (p.e.red == FORGE_RED_CROSS_ENTROPY && live && m < p.M && __ldg(p.target + m) == n) ? v[i] : 0.f;
                        }
                        const int idx = k3_reduce16<2>(mx, se, tl, lane, oa, ob, oc);
                        if ((lane & 1) == 0) { s.red[q][c * 16 + idx] = oa; s.red_s[q][c * 16 + idx] = ob; s.red_t[q][c * 16 + idx] = oc; }
                    } else if (live) {
                        uint16_t *Y = reinterpret_cast<uint16_t *>(p.out);
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            const int m = c * 16 + i;
                            if (m < p.M) Y[(size_t)m * p.N + n] = (uint16_t)(ptx::pack16x2(v[i], 0.f, p.f16) & 0xffffu);
                        }
                    }
                }
            }
            // hand the accumulator back: this warp's reads of it have completed
            ptx::tc_fence_before();
            __syncwarp();
            if (ok && lane == 0) ptx::mbar_arrive(&s.acc_empty[acc]);
            if ((acc ^= 1) == 0) acc_phase ^= 1;

            if (reduce || softmax) {
                k3_epi_sync();
                if (ok && et < p.xr) {
#pragma unroll
                    for (int w = 0; w < K3_EPI_WARPS; ++w) {
                        if (softmax) {
                            lse_merge<false>(running, running_s, s.red[w][et], s.red_s[w][et]);
                            running_t += s.red_t[w][et];
                        } else {
                            running = sum ? running + s.red[w][et] : fmaxf(running, s.red[w][et]);
                        }
                    }
                }
                k3_epi_sync();
            }
        }
        if (!ok) s.abort_flag = 1;

        // ---- fold the CTAs' partials: the last CTA to arrive does it, in a fixed order.  The rows are spread over the
        //      128 threads as (row, chunk of CTAs); chunk results meet in shared memory ----
        if (reduce || softmax) {
            float *out = reinterpret_cast<float *>(p.out);
            float4 *part4 = reinterpret_cast<float4 *>(p.partial);
            if (gridDim.x == 1) {
                if (et < p.M) out[et] = softmax ? running + __logf(running_s) - running_t : running;
            } else {
                if (et < p.xr) {
                    const size_t slot_i = (size_t)blockIdx.x * p.xr + et;
                    if (in_bounds(p.status, BOUNDS_PARTIAL, (long long)slot_i * (softmax ? 4 : 1), softmax ? 4 : 1, p.ws_floats)) {
                        if (softmax) part4[slot_i] = make_float4(running, running_s, running_t, 0.f);
                        else p.partial[slot_i] = running;
                    }
                }
                // one arrival per CTA, by one thread: its release covers the partials the barrier has ordered before it,
                // its acquire (and the next barrier) the other CTAs' partials read below
                k3_epi_sync();
                if (et == 0) s.last_flag = (arrive_acq_rel(&p.counters[0]) == gridDim.x - 1);
                k3_epi_sync();
                if (s.last_flag && !softmax) {
                    // sum / max: a thread takes four rows (one 16-byte load per CTA) of every chunks-th CTA, eight
                    // loads in flight, merged in CTA order (an absent CTA is the neutral element); the chunks'
                    // results meet in shared memory and are merged in chunk order
                    const int quads = p.xr / 4, chunks = K3_EPI_THREADS / quads;       // 32 .. 4 chunks of CTAs
                    const int quad = et % quads, chunk = et / quads;
                    float *ff = &s.fold[0][0];                                          // [chunk][row], at most 512 floats
                    if (chunk < chunks) {
                        float a[4] = {neutral, neutral, neutral, neutral};
                        for (unsigned c0 = chunk; c0 < gridDim.x; c0 += 8 * chunks) {
                            float4 f[8];
#pragma unroll
                            for (int u = 0; u < 8; ++u) {
                                const unsigned c = c0 + u * chunks;
                                f[u] = c < gridDim.x ? __ldcg(&part4[(size_t)c * quads + quad]) : make_float4(neutral, neutral, neutral, neutral);
                            }
#pragma unroll
                            for (int u = 0; u < 8; ++u) {
                                a[0] = sum ? a[0] + f[u].x : fmaxf(a[0], f[u].x);
                                a[1] = sum ? a[1] + f[u].y : fmaxf(a[1], f[u].y);
                                a[2] = sum ? a[2] + f[u].z : fmaxf(a[2], f[u].z);
                                a[3] = sum ? a[3] + f[u].w : fmaxf(a[3], f[u].w);
                            }
                        }
#pragma unroll
                        for (int j = 0; j < 4; ++j) ff[chunk * p.xr + quad * 4 + j] = a[j];
                    }
                    k3_epi_sync();
                    if (et < p.M) {
                        float r = ff[et];
                        for (int j = 1; j < chunks; ++j) r = sum ? r + ff[j * p.xr + et] : fmaxf(r, ff[j * p.xr + et]);
                        out[et] = r;
                    }
                    if (et == 0) p.counters[0] = 0u;
                } else if (s.last_flag) {
                    // softmax statistics: one 16-byte triple per row and CTA
                    const int chunks = K3_EPI_THREADS / p.xr;              // 8 .. 1 chunks of CTAs per row
                    const int row = et % p.xr, chunk = et / p.xr;
                    float mx = -INFINITY, se = 0.f, tl = 0.f;
                    if (chunk < chunks) {
                        for (unsigned c0 = chunk; c0 < gridDim.x; c0 += 8 * chunks) {
                            float4 f[8];
#pragma unroll
                            for (int u = 0; u < 8; ++u) {
                                const unsigned c = c0 + u * chunks;
                                f[u] = c < gridDim.x ? __ldcg(&part4[(size_t)c * p.xr + row]) : make_float4(-INFINITY, 0.f, 0.f, 0.f);
                            }
#pragma unroll
                            for (int u = 0; u < 8; ++u) {
                                lse_merge<false>(mx, se, f[u].x, f[u].y);
                                tl += f[u].z;
                            }
                        }
                    }
                    s.fold[0][et] = mx; s.fold[1][et] = se; s.fold[2][et] = tl;
                    k3_epi_sync();
                    if (et < p.M) {
                        mx = s.fold[0][et]; se = s.fold[1][et]; tl = s.fold[2][et];
                        for (int j = 1; j < chunks; ++j) {
                            lse_merge<false>(mx, se, s.fold[0][j * p.xr + et], s.fold[1][j * p.xr + et]);
                            tl += s.fold[2][j * p.xr + et];
                        }
                        out[et] = mx + __logf(se) - tl;
                    }
                    if (et == 0) p.counters[0] = 0u;
                }
            }
        }
    }

    // ---------------- common exit ----------------
    ptx::tc_fence_before();
    __syncthreads();
    // give-up path only: copies already issued may still be landing in this CTA's shared memory
    if (*(volatile int *)&s.abort_flag) __nanosleep(500000);
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, p.tmem_cols);
    }
}

// ---- host side ---------------------------------------------------------------------------
namespace {
int k3_padded_rows(const forge_fused_linear_desc_t &d) { return (int)((d.M + 15) / 16 * 16); }
uint32_t k3_stage_bytes(int box_groups, int xr, int kb)
{
    const uint32_t wbox = (uint32_t)box_groups * 8 * K3_BK * 2, xbox = (uint32_t)xr * K3_BK * 2;
    const uint32_t boxes = kb * (wbox + xbox), span = (kb - 1) * wbox + K3_A_SPAN;
    return boxes > span ? boxes : span;
}
int k3_stage_count(uint32_t stage)
{
    const int n = (int)(K3_RING_BUDGET / stage);
    return n > K3_MAX_STAGES ? K3_MAX_STAGES : n;
}
// Boxes per stage: what counts is the bytes of W in flight (stages x boxes x box size) and, with two or more boxes,
// that 256 contiguous bytes or more of every row are requested together (measured: at equal bytes in flight two boxes
// beat one by 2-6 %).  A strip of few rows (small N, or N / 8 just above the SM count) has small boxes, and since an MMA
// reads 16 KiB from the start of each -- boxes of one stage may overlap in that span -- only many boxes per stage fill
// the ring: 8 rows of W, one box per stage: 12 KiB in flight; eight boxes: 72 KiB.
int k3_boxes_per_stage(int box_groups, int xr)
{
    if (FORGE_K3_KB != 0) return FORGE_K3_KB;
    const uint32_t wbox = (uint32_t)box_groups * 8 * K3_BK * 2;
    int best = 1;
    double best_score = 0;
    for (int kb = 1; kb <= K3_MAX_KB; ++kb) {
        const int stages = k3_stage_count(k3_stage_bytes(box_groups, xr, kb));
        if (stages < 4 && kb > 1) break;
        const double score = (double)stages * kb * wbox * (kb >= 2 ? 1.0 : 0.9);
        if (score > best_score) { best_score = score; best = kb; }
    }
    return best;
}
uint32_t k3_tmem_cols(int xr)
{
    uint32_t c = 32;
    while (c < 2u * (uint32_t)xr) c <<= 1;
    return c;
}
}  // namespace

forge_status_t k3_plan(const forge_fused_linear_desc_t &d, int sm_count, forge_plan_info_t *info, WorkspaceLayout *wl)
{
    if (d.M > K3_MAX_M || d.N > 0x7fffffff || d.K > 0x7fffffff) return FORGE_ERR_UNSUPPORTED;
    if (d.red == FORGE_RED_LAYERNORM || d.red == FORGE_RED_MEAN_GELU_RESIDUAL) return FORGE_ERR_UNSUPPORTED;
    const int64_t groups = d.N / 8;
    const int grid = (int)(groups < sm_count ? groups : sm_count);
    // strips of equal size, at most 128 rows of W each
    const int64_t per_cta = (groups + grid - 1) / grid;
    const int64_t strips = (per_cta * 8 + K3_MAX_ROWS_W - 1) / K3_MAX_ROWS_W;
    const int box_groups = (int)((per_cta + strips - 1) / strips);
    const int xr = k3_padded_rows(d);
    const int kb = k3_boxes_per_stage(box_groups, xr);
    const uint32_t stage = k3_stage_bytes(box_groups, xr, kb);
    const int stages = k3_stage_count(stage);
    info->kernel = FORGE_KERNEL_BF16_SKINNY;
    info->tile_m = xr;
    info->tile_n = box_groups * 8;
    info->tile_k = kb * K3_BK;
    info->stages = stages;
    info->cluster = 1;
    info->threads = K3_THREADS;
    info->grid = grid;
    info->smem_bytes = (int64_t)(1024 + (size_t)stages * stage + sizeof(K3Smem));
    const bool softmax = d.red == FORGE_RED_LOGSUMEXP || d.red == FORGE_RED_CROSS_ENTROPY;     // float4 partials
    const bool partials = (d.red == FORGE_RED_SUM || d.red == FORGE_RED_MAX || softmax) && grid > 1;
    wl->partial_floats = partials ? (size_t)grid * xr * (softmax ? 4 : 1) : 0;
    wl->counters = partials ? 1 : 0;
    return FORGE_OK;
}

forge_status_t k3_setup(Handle &)
{
    return cudaFuncSetAttribute(k3_bf16_skinny_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)K3_SMEM_LIMIT) == cudaSuccess
               ? FORGE_OK : FORGE_ERR_CUDA;
}

forge_status_t k3_launch(Handle &h, const RunArgs &a)
{
    const forge_fused_linear_desc_t &d = h.d;
    const int xr = h.info.tile_m;
    forge_status_t st;
    if (h.tmX_ptr != a.X) {
        if ((st = encode_tmap_16(&h.tmX, a.X, (uint64_t)d.M, (uint64_t)d.K, (uint32_t)xr, K3_BK, d.dtype == FORGE_F16)) != FORGE_OK) return st;
        h.tmX_ptr = a.X;
    }
    if (h.tmW_ptr != a.W) {
        if ((st = encode_tmap_16(&h.tmW, a.W, (uint64_t)d.N, (uint64_t)d.K, (uint32_t)h.info.tile_n, K3_BK, d.dtype == FORGE_F16)) != FORGE_OK) return st;
        h.tmW_ptr = a.W;
    }
    K3Params p;
    p.f16 = d.dtype == FORGE_F16;
    p.b = (const uint16_t *)a.b;
    p.target = (const int *)a.gamma;
    p.out = a.out;
    p.M = (int)d.M;
    p.N = (int)d.N;
    p.K = (int)d.K;
    p.e = Epilogue{(int)d.act, (int)d.red, d.scale, d.ln_eps, d.has_bias};
    p.partial = h.ws.partial;
    p.counters = h.ws.counters;
    p.status = h.ws.status;
    p.kb = h.info.tile_k / K3_BK;
    p.num_kb = (int)((d.K + h.info.tile_k - 1) / h.info.tile_k);
    p.groups = (int)(d.N / 8);
    p.box_groups = h.info.tile_n / 8;
    p.xr = xr;
    p.stages = h.info.stages;
    p.stage_bytes = k3_stage_bytes(p.box_groups, xr, p.kb);
    p.ring_bytes = (uint32_t)p.stages * p.stage_bytes;
    p.tmem_cols = k3_tmem_cols(xr);
    p.ws_floats = h.ws.partial_floats;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)h.info.grid);
    cfg.blockDim = dim3(K3_THREADS);
    cfg.dynamicSmemBytes = (size_t)h.info.smem_bytes;
    cfg.stream = a.stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, k3_bf16_skinny_kernel, h.tmX, h.tmW, p) == cudaSuccess ? FORGE_OK : FORGE_ERR_CUDA;
}

}  // namespace forge
