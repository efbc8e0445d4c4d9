// K5: fp32 storage, contraction on the 5th-generation tensor cores as three TF32 products.
//
// A TF32 operand keeps the sign, the 8 exponent bits and the upper 10 fraction bits of an fp32
// word.  Every fp32 input is split as x = hi + lo with hi = x with its 13 low fraction bits
// cleared (a TF32 number) and lo = x - hi (exact in fp32; the tensor core keeps its upper 11
// significant bits).  Then
//     x w  =  hi_x hi_w + hi_x lo_w + lo_x hi_w  +  O(2^-21 |x w|),
// three kind::tf32 MMAs per k-step accumulated in fp32 in TMEM, small terms first.  The split
// error is two to three orders of magnitude inside the 1e-4 budget of the fp32 path, at about a
// third of the TF32 tensor rate, which is still several times the FFMA rate of the SMs.
//
// The tensor core adds into its fp32 accumulator with truncation, not rounding to nearest, so
// an accumulator that takes thousands of MMAs drifts towards zero by about 2^-24 per MMA
// (measured: 7e-5 relative at K = 4096 with all 1536 MMAs of an output in one accumulator --
// too close to the 1e-4 budget, and beyond it for same-sign data or larger K).  Therefore an
// accumulator only ever takes one chunk of K (128 by default: 48 MMAs); the epilogue warps
// drain each finished chunk out of TMEM and add it, rounding to nearest, to a running sum they
// keep in registers (128 per thread), while the MMAs of the next chunk fill the other TMEM
// buffer.  The drift is then bounded by the chunk length whatever K is.
//
// Persistent CTA pairs (cluster of two, tcgen05.mma.cta_group::2, 256x256 output tile per pair),
// 512 threads per CTA in four warpgroups with different register shares (setmaxnreg):
//   warp 0        TMA producer: this CTA's 128 rows of the X tile and its 128-row half of the W
//                 tile (128x32 fp32 each, 128-byte swizzle) into a 3-stage ring, completion
//                 counted on the CTA's own "full" barrier;
//   warps 12..15  splitters: wait for the stage, compute lo of every raw word and write it at the
//                 same offset of a second buffer (so the swizzle needs no thought; the raw words
//                 themselves serve as hi, see K5_WRITE_HI), then fence towards the async proxy and
//                 arrive on the leader's "split" barrier;
//   warp 1        MMA issuer (leader CTA, one elected thread): waits for both CTAs' splitters,
//                 issues 3 x 4 MMAs (256x256x8) per stage, commits to the "empty" barriers of
//                 both CTAs and, per chunk of K, to the "accumulator full" barriers;
//   warps 4..11   epilogue, two groups of four warps, one 128-column half of the tile each
//                 (thread <-> output row): per chunk, tcgen05.ld and add to the running sum; after
//                 the last chunk the sum goes back to TMEM and a rolled loop applies bias,
//                 accurate fp32 activation and scale, then stores Y as float4, or forms the row
//                 sum / max / (max, sum exp) / mean chain with per-half-tile partials folded by
//                 the last group to arrive at a row strip.
// TMEM holds two 128x256 fp32 accumulators per CTA, used alternately by the chunks, so the
// draining (and the epilogue of tile i) overlaps the MMAs that follow.  No load is multicast;
// every software wait is bounded.
//
// Last, partly filled wave: when the tiles left over after the full waves are at most half the
// clusters (and at most 8 full waves precede them), each of them is cut along K into S parts of at
// least 512 k that run on S clusters at once.  Parts 1..S-1
// leave their running sums (the registers above) in a scratch area and count themselves in; part 0
// waits for them (bounded), adds them to its own sum in part order and runs the epilogue.  Nothing
// else changes: a part is just a tile with a shorter K range.  A 4096^3 problem (256 tiles on 74
// clusters) takes 3.5 tile times instead of 4.
//
// LayerNorm over N: as on the bf16 kernel, the N-tiles of a row strip are neighbours in the schedule;
// each half tile writes its activated values back to TMEM, publishes (n, mean, M2) per row, waits
// (bounded) for the strip's other half tiles, combines the statistics in part order and normalises
// out of TMEM.  The mean chain publishes gelu(mean) per row and the whole grid writes the residual
// rows at the end.  In both, and with the K cut, CTAs wait on one another: the launch is cooperative.
#include <cmath>
#include <cstring>
#include <mutex>
#include <new>

#include "common.cuh"
#include "epilogue_tmem.cuh"
#include "plan.h"
#include "sm100_ptx.cuh"
#include "tile_schedule.cuh"

namespace forge {

constexpr int K5_BM = 128, K5_BN = 256, K5_BK = 32;     // rows per CTA, columns per pair tile, fp32 per 128-byte row
constexpr int K5_STAGES = 3;
constexpr int K5_THREADS = 512;
constexpr int K5_EPI_WARP0 = 4, K5_SPLIT_WARP0 = 12;
constexpr int K5_EPI_THREADS = 128;
constexpr int K5_SPLIT_WARPS = 4, K5_SPLIT_THREADS = 32 * K5_SPLIT_WARPS;
constexpr uint32_t K5_A_BYTES = K5_BM * K5_BK * 4;                 // 16 KiB: 128 rows of X
constexpr uint32_t K5_B_BYTES = (K5_BN / 2) * K5_BK * 4;           // 16 KiB: this CTA's half of the W tile
constexpr uint32_t K5_RAW_BYTES = K5_A_BYTES + K5_B_BYTES;         // what TMA writes per stage
constexpr uint32_t K5_STAGE_BYTES = 2 * K5_RAW_BYTES;              // raw/hi, then lo
constexpr uint32_t K5_RING_BYTES = K5_STAGES * K5_STAGE_BYTES;     // 192 KiB
constexpr uint32_t K5_TMEM_COLS = 512;
// Tuning builds may override these three (-DFORGE_K5_GROUP_M=.. and so on); the defaults are the measured best.
#ifndef FORGE_K5_K_SERPENTINE
#define FORGE_K5_K_SERPENTINE 1    // 0: every tile walks K upwards
#endif
#ifndef FORGE_K5_GROUP_M
#define FORGE_K5_GROUP_M 16
#endif
#ifndef FORGE_K5_CHUNK_KB
#define FORGE_K5_CHUNK_KB 4
#endif
#ifndef FORGE_K5_TAIL_SPLIT
#define FORGE_K5_TAIL_SPLIT 1      // 0: never cut the last wave's tiles along K
#endif
constexpr int K5_GROUP_M = FORGE_K5_GROUP_M;       // 256-row units per rasterisation group
constexpr int K5_CHUNK_KB = FORGE_K5_CHUNK_KB;     // ring stages (32 k each) accumulated in TMEM before the epilogue drains them
// Register shares after setmaxnreg: the epilogue warpgroups hold a 128-value running sum per
// thread; producer, issuer and splitters need little.  The sum of the shares must not exceed the
// registers the CTA was launched with (checked on the host before the first launch).
constexpr int K5_REGS_EPI = 184, K5_REGS_OTHER = 64;
constexpr int K5_REGS_NEEDED = 256 * K5_REGS_EPI + 256 * K5_REGS_OTHER;
// A kind::tf32 MMA reading a full fp32 word uses its upper 19 bits and ignores the 13 low
// fraction bits (measured on B200: with an identity weight and inputs that run through all 8192
// tail patterns the result is exact, which it would not be if the word were rounded), so the raw
// tile serves as hi.  That is a property of the hardware, not of the instruction set's definition, so it
// is not taken on trust: the first handle created on a device runs a small problem with an identity weight
// whose exact result depends on it (k5_probe_heads); where it does not hold -- or in a build with
// -DK5_WRITE_HI=1 -- the splitters store hi explicitly (words that are TF32 numbers whatever the hardware
// does with low bits) at the price of a third more shared-memory traffic: 717 us instead of 615 us on a
// 4096^3 problem.
#ifndef K5_WRITE_HI
#define K5_WRITE_HI 0
#endif

struct K5Smem {
    uint64_t full[K5_STAGES];       // TMA -> splitters (this CTA)
    uint64_t split[K5_STAGES];      // splitters of both CTAs -> MMA issuer (leader's copy is used)
    uint64_t empty[K5_STAGES];      // MMA -> TMA producer (each CTA)
    uint64_t acc_full[2];
    uint64_t acc_empty[2];
    uint32_t tmem_base;
    int last_flag[2];
    int abort_flag;
    float bias[2][K5_BN];
    float sub[2][K5_BN];            // mean chain: the vector subtracted before the row mean; LayerNorm: gamma
    float beta[2][K5_BN];           // LayerNorm: beta
};
constexpr size_t K5_SMEM_BYTES = 1024 + (size_t)K5_RING_BYTES + sizeof(K5Smem);

struct K5Params {
    const float *b;
    const float *X;             // mean chain only: the residual input
    const void *aux;            // mean chain: sub[N] (float); cross-entropy: target[M] (int32); LayerNorm: gamma[N]
    const float *beta;          // LayerNorm
    unsigned *gen;              // launches whose CTAs wait on one another: run index (see run_index_begin)
    int cooperative;            // CTAs of this launch wait on one another
    void *out;
    int M, N, K;
    Epilogue e;
    float *partial;             // per half tile: [2*tiles_n][M] floats (float4 for the softmax statistics)
    unsigned *counters;         // [tiles_m]
    float *rowg;                // mean chain: gelu(mean) per row, [M]
    unsigned *strips_done;      // mean chain: strips whose rowg values are published; only ever grows: tiles_m per run
    int *status;
    int tiles_m, tiles_n, num_kb;      // tiles_m counts 128-row strips
    int group_m;
    int k_serpentine;           // every other tile of a cluster walks K downwards (see k_serpentine_pays)
    long long ws_floats, ws_counters;   // extents of `partial` and `counters` (bounds-checked build)
    int write_hi;               // the splitters also store the TF32 heads (the raw words do not serve as such here)
    int two_pass;               // LayerNorm of rows with more tiles than CTA pairs: see K5Item::pass
    int chunk_kb;               // stages per TMEM accumulation chunk
    // K split of the last wave's tiles (tail_parts = 1: none)
    int tail_parts;             // S
    int tail_kb;                // k-blocks per part
    float4 *tail_scratch;       // [tail tile][part - 1][rank][column half][32][128] float4
    unsigned *tail_flags;       // [tail tile][rank][column half]; only ever grow: tail_parts - 1 arrivals per run
};

// Item j of this cluster's work list (tile_schedule.cuh): a pair tile (tm = 256-row unit) and a range of k-blocks.
using K5Item = TileItem;
__device__ __forceinline__ bool k5_item(const K5Params &p, int j, int cluster, int clusters, int units_m, K5Item &w)
{
    return schedule_item<false>(j, cluster, clusters, units_m, p.tiles_n, p.num_kb, p.tail_parts, p.tail_kb, p.two_pass != 0, p.group_m, w);
}

template <int N> __device__ __forceinline__ void k5_reg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N> __device__ __forceinline__ void k5_reg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }

__device__ __forceinline__ void k5_epi_bar_sync(int g) { asm volatile("bar.sync %0, %1;" ::"r"(g + 1), "n"(K5_EPI_THREADS) : "memory"); }

__global__ void __launch_bounds__(K5_THREADS, 1)
k5_f32_tf32x3_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW, const K5Params p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *tiles = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    K5Smem &s = *reinterpret_cast<K5Smem *>(tiles + (size_t)K5_RING_BYTES);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = ptx::cluster_ctarank();         // position in the pair; 0 leads
    const int units_m = (p.tiles_m + 1) / 2;              // 256-row units
    const int cluster = (int)(blockIdx.x >> 1), clusters = (int)(gridDim.x >> 1);
    bool ok = true;
    // counters that CTAs wait on only ever grow: this run is complete at `run` times the arrivals of one run
    const unsigned run = p.cooperative ? run_index_begin(p.gen) : 0u;

    if (threadIdx.x == 0) {
        for (int i = 0; i < K5_STAGES; ++i) {
            ptx::mbar_init(&s.full[i], 1);
            ptx::mbar_init(&s.split[i], 2 * K5_SPLIT_WARPS);
            ptx::mbar_init(&s.empty[i], 1);
        }
        for (int i = 0; i < 2; ++i) { ptx::mbar_init(&s.acc_full[i], 1); ptx::mbar_init(&s.acc_empty[i], 16); }
        s.abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tmap(&tmX);
        ptx::prefetch_tmap(&tmW);
    }
    if (warp == 1) {
        ptx::tmem_alloc_pair(&s.tmem_base, K5_TMEM_COLS);
        ptx::tmem_relinquish_pair();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::cluster_sync_all();             // the peer's barriers exist before anything signals them
    ptx::tc_fence_after();
    const uint32_t tmem_base = s.tmem_base;

    if (warp < K5_EPI_WARP0) {
        k5_reg_dec<K5_REGS_OTHER>();          // warpgroup 0: producer, issuer and two idle warps
        if (warp == 0) {
            // ---------------- TMA producer ----------------
            if (ptx::elect_one()) {
                int stage = 0;
                uint32_t phase = 0;
                K5Item w;
                for (int j = 0; ok && k5_item(p, j, cluster, clusters, units_m, w); ++j) {
                    const int tm = 2 * w.tm + (int)rank, tn = w.tn;
                    for (int it = w.kb_lo; it < w.kb_hi; ++it) {
                        const int kb = (p.k_serpentine && (j & 1)) ? w.kb_lo + w.kb_hi - 1 - it : it;
                        if (!ptx::mbar_wait(&s.empty[stage], phase ^ 1, p.status, SITE_STAGE_EMPTY)) { ok = false; break; }
                        if (!in_bounds(p.status, BOUNDS_RING, (long long)stage * K5_STAGE_BYTES, K5_RAW_BYTES, K5_RING_BYTES)) { ok = false; break; }
                        uint8_t *a = tiles + (size_t)stage * K5_STAGE_BYTES;
                        ptx::mbar_expect_tx(&s.full[stage], K5_RAW_BYTES);      // rows past M or N are zero fill and count in full
                        ptx::tma_load_2d(a, &tmX, &s.full[stage], kb * K5_BK, tm * K5_BM);
                        ptx::tma_load_2d(a + K5_A_BYTES, &tmW, &s.full[stage], kb * K5_BK, tn * K5_BN + (int)rank * (K5_BN / 2));
                        if (++stage == K5_STAGES) { stage = 0; phase ^= 1; }
                    }
                }
            }
        } else if (warp == 1) {
            // ---------------- MMA issuer (leader) ----------------
            if (rank == 0 && ptx::elect_one()) {
                const uint32_t idesc = ptx::idesc_tf32_f32(2 * K5_BM, K5_BN);
                int stage = 0, acc = 0;
                uint32_t phase = 0, acc_phase = 0;
                K5Item w;
                for (int j = 0; ok && k5_item(p, j, cluster, clusters, units_m, w); ++j) {
                    for (int kb0 = w.kb_lo; kb0 < w.kb_hi && ok; kb0 += p.chunk_kb) {
                        // one chunk of K into one TMEM buffer, starting from zero
                        if (!ptx::mbar_wait(&s.acc_empty[acc], acc_phase ^ 1, p.status, SITE_ACC_EMPTY)) { ok = false; break; }
                        ptx::tc_fence_after();
                        const uint32_t d_tmem = tmem_base + (uint32_t)acc * K5_BN;
                        if (!in_bounds(p.status, BOUNDS_TMEM, acc * K5_BN, K5_BN, K5_TMEM_COLS)) { ok = false; break; }
                        const int kb1 = min(kb0 + p.chunk_kb, w.kb_hi);
                        for (int kb = kb0; kb < kb1; ++kb) {
                            if (!ptx::mbar_wait(&s.split[stage], phase, p.status, SITE_SPLIT)) { ok = false; break; }
                            if (!in_bounds(p.status, BOUNDS_RING, (long long)stage * K5_STAGE_BYTES, K5_STAGE_BYTES, K5_RING_BYTES)) { ok = false; break; }
                            ptx::tc_fence_after();
                            const uint8_t *a = tiles + (size_t)stage * K5_STAGE_BYTES;
                            const uint64_t a_hi = ptx::smem_desc_k_sw128(a), b_hi = ptx::smem_desc_k_sw128(a + K5_A_BYTES);
                            const uint64_t a_lo = ptx::smem_desc_k_sw128(a + K5_RAW_BYTES);
                            const uint64_t b_lo = ptx::smem_desc_k_sw128(a + K5_RAW_BYTES + K5_A_BYTES);
#pragma unroll
                            for (int k = 0; k < K5_BK / 8; ++k) {     // 8 fp32 = 32 bytes = 2 descriptor units
                                ptx::umma_tf32_pair(d_tmem, a_lo + 2 * k, b_hi + 2 * k, idesc, (kb != kb0) | (k != 0));
                                ptx::umma_tf32_pair(d_tmem, a_hi + 2 * k, b_lo + 2 * k, idesc, 1);
                                ptx::umma_tf32_pair(d_tmem, a_hi + 2 * k, b_hi + 2 * k, idesc, 1);
                            }
                            ptx::umma_commit_pair(&s.empty[stage], 3);
                            if (++stage == K5_STAGES) { stage = 0; phase ^= 1; }
                        }
                        if (!ok) break;
                        ptx::umma_commit_pair(&s.acc_full[acc], 3);
                        if ((acc ^= 1) == 0) acc_phase ^= 1;
                    }
                }
            }
        }
    } else if (warp >= K5_SPLIT_WARP0) {
        // ---------------- splitters ----------------
        k5_reg_dec<K5_REGS_OTHER>();
        const int st = threadIdx.x - 32 * K5_SPLIT_WARP0;   // 0..127
        const uint32_t split_bar[K5_STAGES] = {ptx::mapa_u32(ptx::smem_u32(&s.split[0]), 0),
                                               ptx::mapa_u32(ptx::smem_u32(&s.split[1]), 0),
                                               ptx::mapa_u32(ptx::smem_u32(&s.split[2]), 0)};      // the leader's
        int stage = 0;
        uint32_t phase = 0;
        K5Item w;
        for (int j = 0; ok && k5_item(p, j, cluster, clusters, units_m, w); ++j) {
            for (int kb = w.kb_lo; kb < w.kb_hi; ++kb) {
                if (!ptx::mbar_wait(&s.full[stage], phase, p.status, SITE_TMA_FULL)) { ok = false; break; }
                float4 *raw = reinterpret_cast<float4 *>(tiles + (size_t)stage * K5_STAGE_BYTES);
                float4 *lo = reinterpret_cast<float4 *>(tiles + (size_t)stage * K5_STAGE_BYTES + K5_RAW_BYTES);
                constexpr int PER_THREAD = K5_RAW_BYTES / 16 / K5_SPLIT_THREADS;       // 16 float4
#pragma unroll 8
                for (int i = 0; i < PER_THREAD; ++i) {
                    const int idx = i * K5_SPLIT_THREADS + st;
                    const float4 v = raw[idx];
                    float4 hi;
                    hi.x = __uint_as_float(__float_as_uint(v.x) & 0xffffe000u);
                    hi.y = __uint_as_float(__float_as_uint(v.y) & 0xffffe000u);
                    hi.z = __uint_as_float(__float_as_uint(v.z) & 0xffffe000u);
                    hi.w = __uint_as_float(__float_as_uint(v.w) & 0xffffe000u);
                    lo[idx] = make_float4(v.x - hi.x, v.y - hi.y, v.z - hi.z, v.w - hi.w);
                    if (p.write_hi) raw[idx] = hi;
                }
                ptx::fence_proxy_async_smem();      // these writes are read by the tensor core (async proxy)
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive_cluster(split_bar[stage]);
                if (++stage == K5_STAGES) { stage = 0; phase ^= 1; }
            }
        }
    } else {
        // ---------------- epilogue ----------------
        k5_reg_inc<K5_REGS_EPI>();
        const int q = warp & 3;                       // TMEM lane quarter this warp may read
        const int h = (warp - K5_EPI_WARP0) >> 2;     // column half
        const int et = (threadIdx.x - 32 * K5_EPI_WARP0) & (K5_EPI_THREADS - 1);
        constexpr int HALF = K5_BN / 2, CHUNKS = HALF / 32;
        const int parts = 2 * p.tiles_n;
        int acc = 0;
        uint32_t acc_phase = 0;
        const int red = p.e.red;
        const bool chain = red == FORGE_RED_MEAN_GELU_RESIDUAL;
        const bool ln = red == FORGE_RED_LAYERNORM;
        const bool lse = red == FORGE_RED_LOGSUMEXP || red == FORGE_RED_CROSS_ENTROPY;
        const bool fold = red == FORGE_RED_SUM || red == FORGE_RED_MAX || chain;
        const uint32_t acc_empty_addr[2] = {ptx::mapa_u32(ptx::smem_u32(&s.acc_empty[0]), 0),
                                            ptx::mapa_u32(ptx::smem_u32(&s.acc_empty[1]), 0)};     // the leader's
        int tile_parity = 0;            // bias / sub staging alternates per tile (a slow thread may still read the last one)
        K5Item w;
        for (int j = 0; k5_item(p, j, cluster, clusters, units_m, w); ++j, tile_parity ^= 1) {
            const int tn = w.tn, tm = 2 * w.tm + (int)rank;
            const int m0 = tm * K5_BM, n0 = tn * K5_BN + h * HALF;
            const int part = 2 * tn + h;
            float *sb = s.bias[tile_parity] + h * HALF, *ss = s.sub[tile_parity] + h * HALF;
            {
                const bool in = n0 + et < p.N;
                sb[et] = (p.e.has_bias && in) ? __ldg(p.b + n0 + et) : 0.f;
                if (chain) ss[et] = (in && p.aux) ? __ldg(reinterpret_cast<const float *>(p.aux) + n0 + et) : 0.f;
                if (ln) {
                    ss[et] = in ? __ldg(reinterpret_cast<const float *>(p.aux) + n0 + et) : 0.f;
                    s.beta[tile_parity][h * HALF + et] = in ? __ldg(p.beta + n0 + et) : 0.f;
                }
            }
            const int row = m0 + q * 32 + lane;
            const uint32_t lane_addr = tmem_base + (uint32_t)(h * HALF) + ((uint32_t)(q * 32) << 16);
            if (kDebugBounds && m0 < p.M) {
                // what this group will touch for this tile, checked before any of it is touched (the same verdict in
                // every thread of the group): its tensor-memory columns in both buffers, the strip's counter, the rows
                // of its part in the workspace (one float or one float4 per row), the hand-over area of a K cut
                const bool wide = ln || lse, uses_ws = wide || fold;
                const long long rows = min(K5_BM, p.M - m0), first = (long long)part * p.M + m0;
                bool fine = in_bounds(p.status, BOUNDS_TMEM, K5_BN + h * HALF, HALF, K5_TMEM_COLS);
                if (uses_ws) fine = fine && in_bounds(p.status, BOUNDS_COUNTER, tm, 1, p.ws_counters) &&
                                    in_bounds(p.status, BOUNDS_PARTIAL, wide ? 4 * first : first, wide ? 4 * rows : rows, p.ws_floats);
                if (w.tail >= 0)
                    fine = fine && in_bounds(p.status, BOUNDS_PARTIAL, (long long)(reinterpret_cast<float *>(p.tail_scratch) - p.partial) +
                                             ((((long long)w.tail * (p.tail_parts - 1) + (p.tail_parts - 2)) * 2 + rank) * 2 + h) * (4ll * 32 * K5_EPI_THREADS),
                                             4ll * 32 * K5_EPI_THREADS, p.ws_floats) &&
                           in_bounds(p.status, BOUNDS_COUNTER, (long long)(p.tail_flags - p.counters) + ((long long)w.tail * 2 + rank) * 2 + h, 1, p.ws_counters);
                if (!fine) { ok = false; break; }
            }
            // ---- chunks of K: drain every finished accumulator into the running sum (round to nearest) ----
            float sum[HALF];
#pragma unroll
            for (int j = 0; j < HALF; ++j) sum[j] = 0.f;
            const int nchunks = (w.kb_hi - w.kb_lo + p.chunk_kb - 1) / p.chunk_kb;
            const bool split = w.tail >= 0;           // this item is one of S parts of a tile
            for (int ch = 0; ch < nchunks; ++ch) {
                // the give-up decision must be taken by all threads of the group together
                if (!ptx::mbar_wait(&s.acc_full[acc], acc_phase, p.status, SITE_ACC_FULL)) s.abort_flag = 1;
                k5_epi_bar_sync(h);
                if (*(volatile int *)&s.abort_flag) { ok = false; break; }
                ptx::tc_fence_after();
                const bool last = ch == nchunks - 1;
                if (m0 < p.M && (nchunks > 1 || split)) {
                    const bool put_back = last && !split;      // a split tile's total is formed below
                    const uint32_t ca = lane_addr + (uint32_t)(acc * K5_BN);
#pragma unroll
                    for (int c = 0; c < CHUNKS; ++c) {
                        uint32_t r[32];
                        ptx::tmem_ld_32x32(ca + c * 32, r);
                        ptx::tmem_ld_wait();
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            sum[c * 32 + j] += __uint_as_float(r[j]);
                            r[j] = __float_as_uint(sum[c * 32 + j]);
                        }
                        if (put_back) ptx::tmem_st_32x32(ca + c * 32, r);     // the total goes back for the rolled loop below
                    }
                    if (put_back) ptx::tmem_st_wait();
                }
                if (last) break;                 // this buffer is released after the final pass
                ptx::tc_fence_before();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive_cluster(acc_empty_addr[acc]);
                if ((acc ^= 1) == 0) acc_phase ^= 1;
            }
            if (!ok) break;

            const uint32_t taddr = lane_addr + (uint32_t)(acc * K5_BN);
            if (split && m0 < p.M) {
                // ---- K split of a last-wave tile: parts 1.. hand their sums over, part 0 collects them ----
                unsigned *flag = p.tail_flags + ((size_t)w.tail * 2 + rank) * 2 + h;
                if (w.part > 0) {
                    float4 *dst = p.tail_scratch + ((((size_t)w.tail * (p.tail_parts - 1) + (w.part - 1)) * 2 + rank) * 2 + h) * (32 * K5_EPI_THREADS);
#pragma unroll
                    for (int i = 0; i < HALF / 4; ++i)
                        dst[i * K5_EPI_THREADS + et] = make_float4(sum[4 * i], sum[4 * i + 1], sum[4 * i + 2], sum[4 * i + 3]);
                    k5_epi_bar_sync(h);
                    if (et == 0) arrive_acq_rel(flag);      // its release covers the group's stores, ordered before it by the barrier
                    ptx::tc_fence_before();
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive_cluster(acc_empty_addr[acc]);
                    if ((acc ^= 1) == 0) acc_phase ^= 1;
                    continue;
                }
                if (et == 0 && !wait_counter<100>(flag, run * (unsigned)(p.tail_parts - 1), p.status, SITE_ARRIVAL, w.tail)) s.abort_flag = 1;
                k5_epi_bar_sync(h);
                if (*(volatile int *)&s.abort_flag) { ok = false; break; }
                for (int pp = 1; pp < p.tail_parts; ++pp) {
                    const float4 *src = p.tail_scratch + ((((size_t)w.tail * (p.tail_parts - 1) + (pp - 1)) * 2 + rank) * 2 + h) * (32 * K5_EPI_THREADS);
#pragma unroll
                    for (int i = 0; i < HALF / 4; ++i) {
                        const float4 o = __ldcg(src + i * K5_EPI_THREADS + et);
                        sum[4 * i] += o.x; sum[4 * i + 1] += o.y; sum[4 * i + 2] += o.z; sum[4 * i + 3] += o.w;
                    }
                }
#pragma unroll
                for (int c = 0; c < CHUNKS; ++c) {
                    uint32_t r[32];
#pragma unroll
                    for (int jj = 0; jj < 32; ++jj) r[jj] = __float_as_uint(sum[c * 32 + jj]);
                    ptx::tmem_st_32x32(taddr + c * 32, r);
                }
                ptx::tmem_st_wait();
            }
            if (m0 >= p.M) {
                // this CTA's half of the last pair tile lies past M: nothing to publish
                ptx::tc_fence_before();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive_cluster(acc_empty_addr[acc]);
                if ((acc ^= 1) == 0) acc_phase ^= 1;
                continue;
            }

            if (ln) {
                // ---- LayerNorm over N: row statistics merged across the half tiles of the strip ----
                // sweep 1: activated values back to TMEM, (n, mean, M2) of this half tile by 32-column chunks
                const float *sbe = s.beta[tile_parity] + h * HALF;
                RowStat rs{0.f, 0.f, 0.f};
#pragma unroll 1
                for (int c = 0; c < CHUNKS; ++c) {
                    const int col0 = n0 + c * 32;
                    if (col0 >= p.N) break;
                    uint32_t r[32];
                    ptx::tmem_ld_32x32(taddr + c * 32, r);
                    ptx::tmem_ld_wait();
                    float v[32];
#pragma unroll
                    for (int jj = 0; jj < 32; ++jj) v[jj] = __uint_as_float(r[jj]) + sb[c * 32 + jj];
                    apply_act_array<true>(p.e.act, v, p.e.scale);
#pragma unroll
                    for (int jj = 0; jj < 32; ++jj) r[jj] = __float_as_uint(v[jj]);
                    ptx::tmem_st_32x32(taddr + c * 32, r);
                    rs = merge_stat(rs, chunk_moments(v, min(32, p.N - col0)));
                }
                ptx::tmem_st_wait();
                float4 *stats = reinterpret_cast<float4 *>(p.partial);
                // Rows with more tiles than the grid has CTA pairs cannot all be held on chip at once: every tile is then
                // computed twice.  Pass 0 publishes its triples and moves on (it never waits, so the grid always gets
                // through it); pass 1, which a cluster starts only when it has finished pass 0, recomputes the tile, waits
                // for the strip's triples and normalises.  Twice the arithmetic; the un-normalised tile still never
                // leaves the SM.
                const bool publish = !p.two_pass || w.pass == 0, finish = !p.two_pass || w.pass == 1;
                if (publish && row < p.M) stats[(size_t)part * p.M + row] = make_float4(rs.n, rs.mean, rs.m2, 0.f);
                // publish, then wait (bounded) for the other half tiles of the strip: one arrival per group by one thread
                // (release: the group's triples, ordered before it by the barrier; the acquiring polls and the next
                // barrier make the other groups' triples readable past L1)
                k5_epi_bar_sync(h);
                if (et == 0) {
                    if (publish) arrive_acq_rel(&p.counters[tm]);
                    if (finish && !wait_counter<0>(&p.counters[tm], run * 2u * (unsigned)p.tiles_n, p.status, SITE_ARRIVAL, tm)) s.abort_flag = 1;
                }
                k5_epi_bar_sync(h);
                if (*(volatile int *)&s.abort_flag) { ok = false; break; }
                if (!finish) {
                    ptx::tc_fence_before();
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive_cluster(acc_empty_addr[acc]);
                    if ((acc ^= 1) == 0) acc_phase ^= 1;
                    continue;
                }
                // the strip's parts combined in part order: mean = sum n_i mean_i / sum n_i, M2 = sum (M2_i + n_i (mean_i - mean)^2)
                float rstd = 0.f, shift = 0.f;
                if (row < p.M) shift = -combine_row_moments<true>(stats, parts, p.M, row, p.e.eps, rstd) * rstd;
                // sweep 2: normalise out of TMEM and store
#pragma unroll 1
                for (int c = 0; c < CHUNKS; ++c) {
                    const int col0 = n0 + c * 32;
                    if (col0 >= p.N) break;
                    uint32_t r[32];
                    ptx::tmem_ld_32x32(taddr + c * 32, r);
                    ptx::tmem_ld_wait();
                    if (row < p.M) {
                        const int nv = min(32, p.N - col0);
                        float *dst = reinterpret_cast<float *>(p.out) + (size_t)row * p.N + col0;
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            if (i * 4 < nv) {
                                float y[4];
#pragma unroll
                                for (int jj = 0; jj < 4; ++jj) {
                                    const int cc = c * 32 + i * 4 + jj;
                                    y[jj] = fmaf(fmaf(__uint_as_float(r[i * 4 + jj]), rstd, shift), ss[cc], sbe[cc]);
                                }
                                *reinterpret_cast<float4 *>(dst + i * 4) = make_float4(y[0], y[1], y[2], y[3]);
                            }
                        }
                    }
                }
                ptx::tc_fence_before();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive_cluster(acc_empty_addr[acc]);
                if ((acc ^= 1) == 0) acc_phase ^= 1;
                continue;
            }

            // ---- plain epilogue and the row reductions: one sweep over the half tile (epilogue_tmem.cuh) ----
            const int tgt = (red == FORGE_RED_CROSS_ENTROPY && row < p.M) ? __ldg(reinterpret_cast<const int *>(p.aux) + row) : -1;
            HalfTileRow mine;
            half_tile_sweep<true, CHUNKS>(taddr, n0, p.N, p.e, sb, ss, tgt,
                [&](int col0, const float (&v)[32], int nv) {
                    if (row >= p.M) return;
                    float *dst = reinterpret_cast<float *>(p.out) + (size_t)row * p.N + col0;      // N % 4 == 0: 16-byte aligned
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        if (i * 4 < nv) *reinterpret_cast<float4 *>(dst + i * 4) = make_float4(v[i * 4], v[i * 4 + 1], v[i * 4 + 2], v[i * 4 + 3]);
                }, mine);
            // accumulator drained: hand the TMEM buffer back to the MMA warp
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive_cluster(acc_empty_addr[acc]);
            if (lse || fold)
                strip_fold<true>(p.e, mine, p.partial, part, parts, p.M, p.N, row, et == 0, &p.counters[tm], &s.last_flag[h],
                                 [h] { k5_epi_bar_sync(h); }, reinterpret_cast<float *>(p.out), p.rowg, p.strips_done);
            if ((acc ^= 1) == 0) acc_phase ^= 1;
        }
    }

    // ---------------- mean chain: residual rows ----------------
    // Y[m, :] = X[m, :] + gelu(mean)[m] for all of Y ([M,K]) once every strip has published its
    // values: 2 M K floats of traffic spread over the whole grid instead of being written strip by
    // strip by whichever epilogue group finished a strip (which stalled that CTA's pipeline).
    // CTAs wait on one another here: the launch is cooperative (all CTAs resident) and the wait is bounded.
    if (p.e.red == FORGE_RED_MEAN_GELU_RESIDUAL) {
        if (threadIdx.x == 0 && !wait_counter<200>(p.strips_done, run * (unsigned)p.tiles_m, p.status, SITE_ARRIVAL, (int)blockIdx.x))
            s.abort_flag = 1;
        __syncthreads();
        if (!*(volatile int *)&s.abort_flag) {
            const size_t k4 = (size_t)(p.K >> 2);
            residual_rows<4>(reinterpret_cast<const float4 *>(p.X), reinterpret_cast<float4 *>(p.out), k4, (size_t)p.M * k4,
                          (size_t)blockIdx.x * K5_THREADS + threadIdx.x, (size_t)gridDim.x * K5_THREADS,
                          [&](size_t row) { return __ldcg(p.rowg + row); },
                          [](float4 &x, float g) { x.x += g; x.y += g; x.z += g; x.w += g; });
        } else {
            ok = false;
        }
    }

    // ---------------- teardown ----------------
    if (!ok) __nanosleep(200000);      // give-up path: let copies and MMAs already in flight land
    ptx::tc_fence_before();
    __syncthreads();
    ptx::cluster_sync_all();           // the peer no longer reads this CTA's shared memory or signals its barriers
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc_pair(tmem_base, K5_TMEM_COLS);
    }
    if (p.cooperative && threadIdx.x == 0) run_index_end(p.gen, run);
}

// ---- host side ---------------------------------------------------------------------------
// Grid, K split of the last wave and workspace layout (tile_schedule.cuh).
constexpr int K5_TAIL_MIN_KB = 16;        // a part is worth its hand-over only with 512 k or more
struct K5Layout : ScheduleLayout {
    int64_t grid;
};

static K5Layout k5_layout(const forge_fused_linear_desc_t &d, int sm_count)
{
    const int64_t tiles_m = (d.M + K5_BM - 1) / K5_BM, tiles_n = (d.N + K5_BN - 1) / K5_BN;
    const bool ln = d.red == FORGE_RED_LAYERNORM;
    const bool lse = d.red == FORGE_RED_LOGSUMEXP || d.red == FORGE_RED_CROSS_ENTROPY;
    const bool chain = d.red == FORGE_RED_MEAN_GELU_RESIDUAL;
    const bool fold = d.red == FORGE_RED_SUM || d.red == FORGE_RED_MAX || chain || lse || ln;
    K5Layout L = {};
    // LayerNorm: a tile already waits for its strip; no second dependency, so no K split
    static_cast<ScheduleLayout &>(L) = schedule_layout(
        tiles_m, tiles_n, ((tiles_m + 1) / 2) * tiles_n, sm_count / 2, (int)((d.K + K5_BK - 1) / K5_BK),
        FORGE_K5_TAIL_SPLIT != 0 && !ln, K5_TAIL_MIN_KB,
        fold ? ((lse || ln) ? 4 : 1) * 2 * (size_t)tiles_n * (size_t)d.M : 0, chain, d.M);
    L.grid = 2 * L.ctas;
    return L;
}

forge_status_t k5_plan(const forge_fused_linear_desc_t &d, int sm_count, forge_plan_info_t *info, WorkspaceLayout *wl)
{
    if (d.M > 0x7fffffff || d.N > 0x7fffffff || d.K > 0x7fffffff) return FORGE_ERR_UNSUPPORTED;
    // 16-byte row pitch for TMA (K) and for the float4 stores of Y (N); pairs need two SMs
    if (d.K % 4 != 0 || d.N % 4 != 0 || sm_count < 2) return FORGE_ERR_UNSUPPORTED;
    const K5Layout L = k5_layout(d, sm_count);
    if (L.tiles_m * L.tiles_n > 0x7fffffff) return FORGE_ERR_UNSUPPORTED;
    // (LayerNorm: the tiles of a strip wait for one another; with more of them than CTA pairs every tile is
    // computed twice, see K5Item::pass)
    info->kernel = FORGE_KERNEL_F32_TF32X3;
    info->tile_m = 2 * K5_BM;
    info->tile_n = K5_BN;
    info->tile_k = K5_BK;
    info->stages = K5_STAGES;
    info->cluster = 2;
    info->threads = K5_THREADS;
    info->grid = L.grid;
    info->smem_bytes = (int64_t)K5_SMEM_BYTES;
    wl->partial_floats = L.partial_floats;
    wl->counters = L.counters;
    return FORGE_OK;
}

// CTAs wait on one another in the mean chain (all strips) and in the K split (part 0 on the others).
static bool k5_ctas_wait(const Handle &h)
{
    return h.d.red == FORGE_RED_MEAN_GELU_RESIDUAL || h.d.red == FORGE_RED_LAYERNORM || k5_layout(h.d, h.sm_count).tail_parts > 1;
}

// Do the raw fp32 words serve as TF32 heads on this device, i.e. does a kind::tf32 MMA ignore the 13 low
// fraction bits rather than round them away?  Per device: 0 not known yet, 1 yes, 2 no (heads are written),
// 3 being found out right now (by the nested handle of the probe itself).
static int k5_heads_mode[64];
static std::mutex k5_heads_mutex;

// X = 128 x 32 values whose low 13 fraction bits run through many patterns, W = the first 32 rows of an
// identity (256 x 32), no bias, no activation: Y[:, :32] must reproduce X to 2^-20 if the scheme holds
// (1 * x = hi + lo, of which the tensor core drops at most the two lowest bits of lo); a tensor core that
// rounded the raw word to the nearest TF32 number instead would be off by up to 2^-11 |x| on about half of them.
static forge_status_t k5_probe_heads(int device, int *mode)
{
    constexpr int M = 128, N = 256, K = 32;
    float *hx = new (std::nothrow) float[M * K + N * K + M * N];
    if (!hx) return FORGE_ERR_ALLOC;
    float *hw = hx + M * K, *hy = hw + N * K;
    for (int i = 0; i < M * K; ++i) {
        const uint32_t tail = ((uint32_t)i * 2654435761u) & 0x1fffu, head = ((uint32_t)i * 40503u) & 0x3ffu;
        const uint32_t bits = ((uint32_t)(120 + i % 16) << 23) | (head << 13) | tail | (((uint32_t)i & 1u) << 31);
        std::memcpy(&hx[i], &bits, 4);
    }
    for (int i = 0; i < N * K; ++i) hw[i] = (i / K == i % K) ? 1.0f : 0.0f;
    forge_fused_linear_desc_t d = {};
    d.M = M; d.N = N; d.K = K;
    d.dtype = FORGE_F32_TF32X3; d.act = FORGE_ACT_IDENTITY; d.red = FORGE_RED_NONE;
    d.scale = 1.0f; d.ln_eps = 0.f; d.has_bias = 0; d.device = device;
    float *dx = nullptr;
    forge_fused_linear_t probe = nullptr;
    forge_status_t st = cudaMalloc(&dx, sizeof(float) * (M * K + N * K + M * N)) == cudaSuccess ? FORGE_OK : FORGE_ERR_ALLOC;
    if (st == FORGE_OK) st = forge_fused_linear_create(&d, &probe);
    if (st == FORGE_OK && cudaMemcpy(dx, hx, sizeof(float) * (M * K + N * K), cudaMemcpyHostToDevice) != cudaSuccess) st = FORGE_ERR_CUDA;
    if (st == FORGE_OK) st = forge_fused_linear_run(probe, dx, dx + M * K, nullptr, nullptr, nullptr, dx + M * K + N * K, nullptr);
    if (st == FORGE_OK) st = forge_fused_linear_last_status(probe);
    if (st == FORGE_OK && cudaMemcpy(hy, dx + M * K + N * K, sizeof(float) * M * N, cudaMemcpyDeviceToHost) != cudaSuccess) st = FORGE_ERR_CUDA;
    if (st == FORGE_OK) {
        bool holds = true;
        for (int m = 0; m < M && holds; ++m)
            for (int k = 0; k < K; ++k) {
                const float x = hx[m * K + k], y = hy[m * N + k];
                if (!(std::fabs(y - x) <= std::fabs(x) * (1.0f / 262144.0f))) { holds = false; break; }      // 2^-18
            }
        *mode = holds ? 1 : 2;
    }
    if (probe) forge_fused_linear_destroy(probe);
    if (dx) cudaFree(dx); else cudaGetLastError();
    delete[] hx;
    return st;
}

forge_status_t k5_setup(Handle &h)
{
    if (h.d.device >= 64) return FORGE_ERR_UNSUPPORTED;
    {
        std::unique_lock<std::mutex> lock(k5_heads_mutex);
        if (K5_WRITE_HI) k5_heads_mode[h.d.device] = 2;
        if (k5_heads_mode[h.d.device] == 0) {
            k5_heads_mode[h.d.device] = 3;
            lock.unlock();                       // the probe creates a handle of its own, which comes through here
            int mode = 0;
            const forge_status_t st = k5_probe_heads(h.d.device, &mode);
            lock.lock();
            k5_heads_mode[h.d.device] = st == FORGE_OK ? mode : 0;
            if (st != FORGE_OK) return st;
        }
    }
    // setmaxnreg.inc waits until the registers it asks for are free: the shares must fit into what
    // a CTA is launched with, or the kernel is never launched
    cudaFuncAttributes fa;
    if (cudaFuncGetAttributes(&fa, k5_f32_tf32x3_kernel) != cudaSuccess || fa.numRegs * K5_THREADS < K5_REGS_NEEDED)
        return FORGE_ERR_CUDA;
    if (cudaFuncSetAttribute(k5_f32_tf32x3_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)K5_SMEM_BYTES) != cudaSuccess)
        return FORGE_ERR_CUDA;
    if (k5_ctas_wait(h)) {
        // CTAs that wait on one another must all be resident at once
        int coop = 0, per_sm = 0;
        if (cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, h.d.device) != cudaSuccess || !coop) return FORGE_ERR_CUDA;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k5_f32_tf32x3_kernel, K5_THREADS, K5_SMEM_BYTES) != cudaSuccess ||
            (int64_t)per_sm * h.sm_count < h.info.grid)
            return FORGE_ERR_CUDA;
    }
    return FORGE_OK;
}

forge_status_t k5_launch(Handle &h, const RunArgs &a)
{
    const forge_fused_linear_desc_t &d = h.d;
    forge_status_t st;
    if (h.tmX_ptr != a.X) {
        if ((st = encode_tmap_f32(&h.tmX, a.X, (uint64_t)d.M, (uint64_t)d.K, K5_BM, K5_BK)) != FORGE_OK) return st;
        h.tmX_ptr = a.X;
    }
    if (h.tmW_ptr != a.W) {
        if ((st = encode_tmap_f32(&h.tmW, a.W, (uint64_t)d.N, (uint64_t)d.K, K5_BN / 2, K5_BK)) != FORGE_OK) return st;
        h.tmW_ptr = a.W;
    }
    K5Params p = {};
    p.b = (const float *)a.b;
    p.X = (const float *)a.X;
    p.aux = a.gamma;
    p.out = a.out;
    p.M = (int)d.M;
    p.N = (int)d.N;
    p.K = (int)d.K;
    p.e = Epilogue{(int)d.act, (int)d.red, d.scale, d.ln_eps, d.has_bias};
    p.partial = h.ws.partial;
    p.counters = h.ws.counters;
    p.status = h.ws.status;
    p.tiles_m = (int)((d.M + K5_BM - 1) / K5_BM);
    const K5Layout L = k5_layout(d, h.sm_count);
    p.gen = h.ws.counters + L.gen_idx;
    p.ws_floats = h.ws.partial_floats;
    p.ws_counters = h.ws.counter_words;
    p.write_hi = k5_heads_mode[d.device] == 2;
    p.two_pass = d.red == FORGE_RED_LAYERNORM && L.tiles_n > L.grid / 2;
    p.cooperative = k5_ctas_wait(h);
    p.rowg = h.ws.partial + L.rowg_off;
    p.strips_done = h.ws.counters + L.strips_done_idx;
    p.tail_parts = L.tail_parts;
    p.tail_kb = L.tail_kb;
    p.tail_scratch = reinterpret_cast<float4 *>(h.ws.partial + L.scratch_off);
    p.tail_flags = h.ws.counters + L.tail_flags_idx;
    p.beta = (const float *)a.beta;
    p.tiles_n = (int)((d.N + K5_BN - 1) / K5_BN);
    p.num_kb = (int)((d.K + K5_BK - 1) / K5_BK);
    p.group_m = d.red == FORGE_RED_LAYERNORM ? 0 : K5_GROUP_M;
    p.chunk_kb = K5_CHUNK_KB;
    p.k_serpentine = FORGE_K5_K_SERPENTINE && k_serpentine_pays(d, h.info.grid / 2, 2 * K5_BM, K5_BN, p.group_m * 2 * K5_BM, 4, h.l2_bytes);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)h.info.grid);
    cfg.blockDim = dim3(K5_THREADS);
    cfg.dynamicSmemBytes = K5_SMEM_BYTES;
    cfg.stream = a.stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (p.cooperative && cooperative_launch_enabled()) {
        attr[1].id = cudaLaunchAttributeCooperative;
        attr[1].val.cooperative = 1;
        cfg.numAttrs = 2;
    }
    return cudaLaunchKernelEx(&cfg, k5_f32_tf32x3_kernel, h.tmX, h.tmW, p) == cudaSuccess ? FORGE_OK : FORGE_ERR_CUDA;
}

}  // namespace forge
