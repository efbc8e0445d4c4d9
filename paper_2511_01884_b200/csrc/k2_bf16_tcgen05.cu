// K2: bf16 fused linear on the 5th-generation tensor cores.
//
// Persistent, warp-specialised CTA (one per SM):
//   warp 0      TMA producer: X and W tiles (128x64 and 256x64 bf16, 128-byte swizzle) into a
//               4-stage shared-memory ring, completion counted in bytes on "full" mbarriers;
//   warp 1      MMA issuer: one elected thread issues tcgen05.mma (128x256x16, fp32 accumulate
//               in TMEM); tcgen05.commit releases ring stages and publishes finished tiles;
//   warps 2..9  epilogue, two groups of four warps, each owning one 128-column half of every
//               tile: tcgen05.ld of the accumulator (thread <-> output row), bias, activation,
//               scale, then either bf16 stores of Y or the row sum / max.
// TMEM holds two 128x256 fp32 accumulators, so the epilogue of tile i overlaps the MMAs of
// tile i+1.  No load is multicast; every wait is bounded (see ptx::mbar_wait).
//
// K4 (LayerNorm over N) is the same kernel with a different tile order and epilogue: the
// N-tiles of one 128-row strip are consecutive tiles, hence run on different SMs at about
// the same time.  Each epilogue group makes one sweep over its half of the accumulator (bias,
// activation, scale, per-row (n, mean, M2) of its 128 columns), keeps the activated values in
// registers (128 per thread; the epilogue warpgroups take a larger register share with
// setmaxnreg, which is why this form runs 384 threads: warpgroup 0 = producer, issuer and two idle
// warps) and hands the TMEM buffer back at once.  It then publishes the row triples to a small
// workspace, waits -- bounded -- until the strip's other tiles have published theirs, merges the
// triples in tile order (Chan et al.), normalises the registers and stores.  Only the 16-byte
// triples travel through global memory; the un-normalised tile never leaves the SM.  The wait
// costs the tensor cores nothing as long as it is shorter than two tiles: the MMAs of the next
// two tiles have both TMEM buffers to go to.  CTAs wait on one another, so the launch is
// cooperative and a strip may not have more tiles than there are CTAs.
#include "common.cuh"
#include "epilogue_tmem.cuh"
#include "plan.h"
#include "sm100_ptx.cuh"
#include "tile_schedule.cuh"

namespace forge {

constexpr int K2_BM = 128, K2_BN = 256, K2_BK = 64;
constexpr int K2_MAX_STAGES = 6;
constexpr int K2_EPI_THREADS = 128;
// Threads per CTA and first epilogue warp.  Plain form: TMA warp, MMA warp, 2 x 4 epilogue warps.  LayerNorm:
// warpgroup 0 = TMA warp, MMA warp and two idle warps, warpgroups 1 and 2 = the two epilogue groups, so that
// setmaxnreg (a warpgroup-wide instruction) can move registers from the former to the latter.
template <bool LN> struct K2Shape {
    static constexpr int THREADS = LN ? 384 : 320;
    static constexpr int EPI_WARP0 = LN ? 4 : 2;
};
// LayerNorm register shares: 128 x 40 + 256 x 232 = 64512 = 384 x 168, what the CTA is launched with
// (checked on the host before the first launch: setmaxnreg.inc waits for ever for registers that are not there).
constexpr int K4_REGS_EPI = 232, K4_REGS_OTHER = 40;
constexpr int K4_REGS_NEEDED = 128 * K4_REGS_OTHER + 256 * K4_REGS_EPI;
constexpr uint32_t K2_A_BYTES = K2_BM * K2_BK * 2;
constexpr uint32_t K2_TMEM_COLS = 512;
// Shared-memory ring.  One CTA per tile: a stage holds the 128-row X tile and the 256-row W tile
// (48 KiB, 4 stages).  CTA pair (cta_group::2, 256x256 tile per pair): each CTA holds its own
// 128 rows of X and its 128-row half of the W tile (32 KiB, 6 stages); the tensor cores of both
// SMs read each half once.
template <bool PAIR> struct K2Ring {
    static constexpr uint32_t B_BYTES = (PAIR ? K2_BN / 2 : K2_BN) * K2_BK * 2;
    static constexpr uint32_t STAGE_BYTES = K2_A_BYTES + B_BYTES;
    static constexpr int STAGES = PAIR ? 6 : 4;
    static constexpr uint32_t BYTES = STAGES * STAGE_BYTES;      // 192 KiB either way
};
// Tuning builds may override these three (-DFORGE_K2_GROUP_M=.. and so on); the defaults are the measured best.
#ifndef FORGE_K2_GROUP_M
#define FORGE_K2_GROUP_M 32
#endif
#ifndef FORGE_K2_K_SERPENTINE
#define FORGE_K2_K_SERPENTINE 1    // 0: every tile walks K upwards
#endif
#ifndef FORGE_K2_PAIR
#define FORGE_K2_PAIR 1            // 0: one CTA per tile, never CTA pairs
#endif
#ifndef FORGE_K2_TAIL_SPLIT
#define FORGE_K2_TAIL_SPLIT 1      // 0: never cut the last wave's tiles along K
#endif
constexpr int K2_GROUP_M = FORGE_K2_GROUP_M;      // 128-row tiles per rasterisation group (keeps a wave's operands in L2)

struct K2Smem {
    uint64_t full[K2_MAX_STAGES];
    uint64_t empty[K2_MAX_STAGES];
    uint64_t acc_full[2];
    uint64_t acc_empty[2];
    uint32_t tmem_base;
    int last_flag[2];
    int abort_flag;
    uint4 store_patch[8][128];  // 2 KiB per epilogue warp: see k2_store_row_pieces
    float bias[2][K2_BN];
    float gamma[2][K2_BN];
    float beta[2][K2_BN];
};
// One CTA per tile with at most 64 rows of X: the X box is 64 rows (8 KiB), which makes room for a fifth stage
// (5 x 40 KiB): these problems are bound by the stream of W, and what counts is the bytes in flight.  The MMA
// still spans 128 rows; rows 64..127 of its A operand are the first rows of the stage's W tile (finite values),
// and the accumulator rows they produce are never read.
constexpr uint32_t K2_A_BYTES_SHORT = K2_A_BYTES / 2;
constexpr int K2_STAGES_SHORT = 5;
constexpr size_t K2_RING_BYTES = (size_t)K2_STAGES_SHORT * (K2_A_BYTES_SHORT + K2Ring<false>::B_BYTES);     // 200 KiB, the largest
static_assert(K2Ring<false>::BYTES <= K2_RING_BYTES && K2Ring<true>::BYTES <= K2_RING_BYTES && K2_STAGES_SHORT <= K2_MAX_STAGES, "ring");
constexpr size_t K2_SMEM_BYTES = 1024 + K2_RING_BYTES + sizeof(K2Smem);
static_assert(K2_SMEM_BYTES <= 227 * 1024, "shared memory of one CTA");

struct K2Params {
    int f16;                    // storage format of X, W, b, gamma, beta, Y: IEEE half (1) or bfloat16 (0)
    const uint16_t *b;
    const uint16_t *X;          // mean chain only: the residual input
    void *out;
    int M, N, K;
    Epilogue e;
    const uint16_t *gamma, *beta;
    float *partial;       // per half tile: sum/max [2*tiles_n][M] floats; layernorm [2*tiles_n][M] float4 triples
    unsigned *counters;   // [tiles_m]
    int *status;
    int tiles_m, tiles_n, num_kb;      // tiles_m counts 128-row strips
    int group_m;          // row units per rasterisation group
    unsigned *gen;        // launches whose CTAs wait on one another: run index (see run_index_begin)
    int two_pass;         // LayerNorm of rows with more tiles than CTAs (pairs): see K2Item::pass
    int short_x;          // one CTA per tile and M <= 64: 64-row X box, five stages
    int k_serpentine;     // every other tile of a unit walks K downwards (a wave's operands exceed half of L2)
    long long ws_floats, ws_counters;      // extents of `partial` and `counters` (bounds-checked build)
    // K split of the last wave's tiles (tail_parts = 1: none)
    int tail_parts;           // S
    int tail_kb;              // k-blocks per part
    float4 *tail_scratch;     // [tail tile][part - 1][rank][column half][32][128] float4: raw accumulators
    unsigned *tail_flags;     // [tail tile][rank][column half]; only ever grow: tail_parts - 1 arrivals per run
    int cooperative;          // CTAs of this launch wait on one another
    float *rowg;              // mean chain: gelu(mean) per row, [M]
    unsigned *strips_done;    // mean chain: strips whose rowg values are published; only ever grows: tiles_m per run
};

// Item j of this unit's work list (tile_schedule.cuh).  LayerNorm: the N-tiles of a strip are neighbours in the
// schedule (group_m = 0) and rows wider than the grid take every tile twice.
using K2Item = TileItem;
template <bool LN>
__device__ __forceinline__ bool k2_item(const K2Params &p, int j, int unit, int units, int unit_rows, K2Item &w)
{
    return schedule_item<true>(j, unit, units, unit_rows, p.tiles_n, p.num_kb, p.tail_parts, p.tail_kb, LN && p.two_pass,
                               LN ? 0 : p.group_m, w);
}

// 32 columns of Y for the 32 rows of a warp (thread <-> row, four 16-byte pieces each) -> global memory through a
// 2-KiB patch of shared memory, so that one store instruction writes 8 rows x 64 contiguous bytes (whole sectors)
// instead of 32 rows x 16 bytes.  Piece i of row r lies at slot i ^ ((r >> 1) & 3) of the row's 64 bytes: both the
// row-wise writes and the transposed reads are free of bank conflicts.  row0 = the warp's first row.
__device__ __forceinline__ void k2_store_row_pieces(uint4 *patch, int lane, const uint4 (&w4)[4], __nv_bfloat16 *out,
                                                    int row0, int M, int N, int col0)
{
#pragma unroll
    for (int i = 0; i < 4; ++i) patch[lane * 4 + (i ^ ((lane >> 1) & 3))] = w4[i];
    __syncwarp();
    const int piece = lane & 3, col = col0 + piece * 8;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int r = 8 * i + (lane >> 2), row = row0 + r;
        const uint4 x = patch[r * 4 + (piece ^ ((r >> 1) & 3))];
        if (row < M && col < N) *reinterpret_cast<uint4 *>(out + (size_t)row * N + col) = x;      // N % 8 == 0: whole pieces
    }
    __syncwarp();          // the patch is free for the next 32 columns
}

// named barrier of epilogue group g (ids 1 and 2; 0 is __syncthreads)
__device__ __forceinline__ void epi_bar_sync(int g) { asm volatile("bar.sync %0, %1;" ::"r"(g + 1), "n"(K2_EPI_THREADS) : "memory"); }

// PAIR: the kernel runs as clusters of two CTAs on one TPC.  A pair owns a 256x256 output tile:
// CTA `rank` loads rows [128 rank, 128 rank + 128) of the X tile and of the W tile; the leader
// (rank 0) issues tcgen05.mma.cta_group::2, which accumulates 128 rows x 256 columns in the TMEM
// of each CTA; each CTA runs the epilogue of its own 128 rows.  Barriers: both CTAs' loads are
// credited to the leader's "full" barrier, tcgen05.commit signals the "empty" and "accumulator
// full" barriers of both CTAs, the epilogues of both CTAs arrive on the leader's "accumulator
// empty" barrier.
template <bool LN, bool PAIR>
__global__ void __launch_bounds__(K2Shape<LN>::THREADS, 1)
k2_bf16_tcgen05_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW, const K2Params p)
{
    using Ring = K2Ring<PAIR>;
    const bool short_x = !PAIR && p.short_x;
    const int STAGES = short_x ? K2_STAGES_SHORT : Ring::STAGES;
    const uint32_t A_BYTES = short_x ? K2_A_BYTES_SHORT : K2_A_BYTES, STAGE_BYTES = A_BYTES + Ring::B_BYTES;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *tiles = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    K2Smem &s = *reinterpret_cast<K2Smem *>(tiles + K2_RING_BYTES);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = PAIR ? ptx::cluster_ctarank() : 0u;        // position in the pair; 0 leads
    // work units: tiles (one CTA each) or 256-row pair tiles (one cluster each)
    const int unit_rows = PAIR ? (p.tiles_m + 1) / 2 : p.tiles_m;
    const int unit = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;       // this CTA's (pair's) place among ...
    const int units = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;        // ... the units that share the work
    bool ok = true;
    // counters that CTAs wait on only ever grow: this run is complete at `run` times the arrivals of one run
    const unsigned run = p.cooperative ? run_index_begin(p.gen) : 0u;

    if (threadIdx.x == 0) {
        for (int i = 0; i < K2_MAX_STAGES; ++i) { ptx::mbar_init(&s.full[i], 1); ptx::mbar_init(&s.empty[i], 1); }
        for (int i = 0; i < 2; ++i) { ptx::mbar_init(&s.acc_full[i], 1); ptx::mbar_init(&s.acc_empty[i], PAIR ? 16 : 8); }
        s.abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tmap(&tmX);
        ptx::prefetch_tmap(&tmW);
    }
    if (warp == 1) {
        if (PAIR) {
            ptx::tmem_alloc_pair(&s.tmem_base, K2_TMEM_COLS);
            ptx::tmem_relinquish_pair();
        } else {
            ptx::tmem_alloc(&s.tmem_base, K2_TMEM_COLS);
            ptx::tmem_relinquish();
        }
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (PAIR) ptx::cluster_sync_all();       // the peer's barriers exist before anything signals them
    ptx::tc_fence_after();
    const uint32_t tmem_base = s.tmem_base;

    constexpr int EPI_WARP0 = K2Shape<LN>::EPI_WARP0, THREADS = K2Shape<LN>::THREADS;
    // LayerNorm: warpgroup 0 hands registers to the epilogue warpgroups (each warp of a warpgroup executes its own
    // setmaxnreg; the compiler sizes the code that follows each one accordingly)
    if (LN && warp < EPI_WARP0) asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(K4_REGS_OTHER));
    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (ptx::elect_one()) {
            int stage = 0;
            uint32_t phase = 0;
            K2Item w;
            for (int j = 0; ok && k2_item<LN>(p, j, unit, units, unit_rows, w); ++j) {
                const int tm = PAIR ? 2 * w.tm + (int)rank : w.tm, tn = w.tn;
                for (int it = w.kb_lo; it < w.kb_hi; ++it) {
                    // K serpentine (see k2_k_serpentine)
                    const int kb = (p.k_serpentine && (j & 1)) ? w.kb_lo + w.kb_hi - 1 - it : it;
                    if (!ptx::mbar_wait(&s.empty[stage], phase ^ 1, p.status, SITE_STAGE_EMPTY)) { ok = false; break; }
                    if (!in_bounds(p.status, BOUNDS_RING, (long long)stage * STAGE_BYTES, STAGE_BYTES, (long long)K2_RING_BYTES)) { ok = false; break; }
                    uint8_t *a = tiles + (size_t)stage * STAGE_BYTES;
                    if (PAIR) {
                        // the leader's barrier counts the bytes of both CTAs (rows past M or N are zero fill
                        // and count in full)
                        if (rank == 0) ptx::mbar_expect_tx(&s.full[stage], 2 * STAGE_BYTES);
                        const uint32_t bar = ptx::mapa_u32(ptx::smem_u32(&s.full[stage]), 0);
                        ptx::tma_load_2d_pair(a, &tmX, bar, kb * K2_BK, tm * K2_BM);
                        ptx::tma_load_2d_pair(a + A_BYTES, &tmW, bar, kb * K2_BK, tn * K2_BN + (int)rank * (K2_BN / 2));
                    } else {
                        ptx::mbar_expect_tx(&s.full[stage], STAGE_BYTES);
                        ptx::tma_load_2d(a, &tmX, &s.full[stage], kb * K2_BK, tm * K2_BM);
                        ptx::tma_load_2d(a + A_BYTES, &tmW, &s.full[stage], kb * K2_BK, tn * K2_BN);
                    }
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if ((!PAIR || rank == 0) && ptx::elect_one()) {
            const uint32_t idesc = ptx::idesc_16_f32(PAIR ? 2 * K2_BM : K2_BM, K2_BN, p.f16);
            int stage = 0, acc = 0;
            uint32_t phase = 0, acc_phase = 0;
            K2Item w;
            for (int j = 0; ok && k2_item<LN>(p, j, unit, units, unit_rows, w); ++j) {
                if (!ptx::mbar_wait(&s.acc_empty[acc], acc_phase ^ 1, p.status, SITE_ACC_EMPTY)) { ok = false; break; }
                ptx::tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)acc * K2_BN;
                if (!in_bounds(p.status, BOUNDS_TMEM, acc * K2_BN, K2_BN, K2_TMEM_COLS)) { ok = false; break; }
                for (int kb = w.kb_lo; kb < w.kb_hi; ++kb) {
                    if (!ptx::mbar_wait(&s.full[stage], phase, p.status, SITE_TMA_FULL)) { ok = false; break; }
                    if (!in_bounds(p.status, BOUNDS_RING, (long long)stage * STAGE_BYTES, STAGE_BYTES, (long long)K2_RING_BYTES)) { ok = false; break; }
                    ptx::tc_fence_after();
                    const uint8_t *a = tiles + (size_t)stage * STAGE_BYTES;
                    const uint64_t adesc = ptx::smem_desc_k_sw128(a);
                    const uint64_t bdesc = ptx::smem_desc_k_sw128(a + A_BYTES);
#pragma unroll
                    for (int k = 0; k < K2_BK / 16; ++k) {     // 16 bf16 = 32 bytes = 2 descriptor units
                        if (PAIR) ptx::umma_bf16_pair(d_tmem, adesc + 2 * k, bdesc + 2 * k, idesc, (kb != w.kb_lo) | (k != 0));
                        else ptx::umma_bf16(d_tmem, adesc + 2 * k, bdesc + 2 * k, idesc, (kb != w.kb_lo) | (k != 0));
                    }
                    if (PAIR) ptx::umma_commit_pair(&s.empty[stage], 3);
                    else ptx::umma_commit(&s.empty[stage]);
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
                if (!ok) break;
                if (PAIR) ptx::umma_commit_pair(&s.acc_full[acc], 3);
                else ptx::umma_commit(&s.acc_full[acc]);
                if ((acc ^= 1) == 0) acc_phase ^= 1;
            }
        }
    } else if (warp >= EPI_WARP0) {
        // ---------------- epilogue ----------------
        if (LN) asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(K4_REGS_EPI));
        // Two independent groups of four warps; group h owns columns [128h, 128h+128) of every
        // tile ("part" 2*tn + h of the row strip) and has its own named barrier.
        const int q = warp & 3;                       // TMEM lane quarter this warp may read
        const int h = (warp - EPI_WARP0) >> 2;        // column half
        const int et = (threadIdx.x - 32 * EPI_WARP0) & (K2_EPI_THREADS - 1);     // 0..127 inside the group
        constexpr int HALF = K2_BN / 2, CHUNKS = HALF / 32;
        const int parts = 2 * p.tiles_n;
        int acc = 0;
        uint32_t acc_phase = 0;
        const bool chain = p.e.red == FORGE_RED_MEAN_GELU_RESIDUAL;       // subtract, row mean, GELU, residual add
        const bool reduce = p.e.red == FORGE_RED_SUM || p.e.red == FORGE_RED_MAX || chain;
        const uint32_t acc_empty_addr[2] = {ptx::mapa_u32(ptx::smem_u32(&s.acc_empty[0]), 0),
                                            ptx::mapa_u32(ptx::smem_u32(&s.acc_empty[1]), 0)};   // the leader's (PAIR)
        K2Item w;
        for (int j = 0; k2_item<LN>(p, j, unit, units, unit_rows, w); ++j) {
            const int tm = PAIR ? 2 * w.tm + (int)rank : w.tm, tn = w.tn;
            const int m0 = tm * K2_BM, n0 = tn * K2_BN + h * HALF;
            const int part = 2 * tn + h;
            float *sb = s.bias[acc] + h * HALF, *sg = s.gamma[acc] + h * HALF, *sbe = s.beta[acc] + h * HALF;
            // bias (and gamma, beta) of this half tile -> shared memory as fp32, one value per thread
            {
                const bool in = n0 + et < p.N;
                sb[et] = (p.e.has_bias && in) ? ptx::load16(p.b, n0 + et, p.f16) : 0.f;
                if (LN) {
                    sg[et] = in ? ptx::load16(p.gamma, n0 + et, p.f16) : 0.f;
                    sbe[et] = in ? ptx::load16(p.beta, n0 + et, p.f16) : 0.f;
                } else if (chain) {          // the vector subtracted before the row mean
                    sg[et] = (in && p.gamma) ? ptx::load16(p.gamma, n0 + et, p.f16) : 0.f;
                }
            }
            // the give-up decision must be taken by all threads of the group together
            if (!ptx::mbar_wait(&s.acc_full[acc], acc_phase, p.status, SITE_ACC_FULL)) s.abort_flag = 1;
            epi_bar_sync(h);
            if (*(volatile int *)&s.abort_flag) { ok = false; break; }
            ptx::tc_fence_after();

            const int row = m0 + q * 32 + lane;
            const uint32_t taddr = tmem_base + (uint32_t)(acc * K2_BN + h * HALF) + ((uint32_t)(q * 32) << 16);
            if (kDebugBounds && m0 < p.M) {
                // what this group will touch for this tile, checked before any of it is touched (the same verdict in
                // every thread of the group): its tensor-memory columns, the strip's counter, the rows of its part
                // in the workspace (one float or one float4 per row), the hand-over area of a K cut
                const bool wide = LN || p.e.red == FORGE_RED_LOGSUMEXP || p.e.red == FORGE_RED_CROSS_ENTROPY;
                const bool uses_ws = LN || reduce || wide;
                const long long rows = min(K2_BM, p.M - m0), first = (long long)part * p.M + m0;
                bool fine = in_bounds(p.status, BOUNDS_TMEM, acc * K2_BN + h * HALF, HALF, K2_TMEM_COLS);
                if (uses_ws) fine = fine && in_bounds(p.status, BOUNDS_COUNTER, tm, 1, p.ws_counters) &&
                                    in_bounds(p.status, BOUNDS_PARTIAL, wide ? 4 * first : first, wide ? 4 * rows : rows, p.ws_floats);
                if (!LN && w.tail >= 0)
                    fine = fine && in_bounds(p.status, BOUNDS_PARTIAL, (long long)(reinterpret_cast<float *>(p.tail_scratch) - p.partial) +
                                             ((((long long)w.tail * (p.tail_parts - 1) + (p.tail_parts - 2)) * 2 + rank) * 2 + h) * (4ll * 32 * K2_EPI_THREADS),
                                             4ll * 32 * K2_EPI_THREADS, p.ws_floats) &&
                           in_bounds(p.status, BOUNDS_COUNTER, (long long)(p.tail_flags - p.counters) + ((long long)w.tail * 2 + rank) * 2 + h, 1, p.ws_counters);
                if (!fine) { ok = false; break; }
            }
            if (PAIR && m0 >= p.M) {
                // second half of the last pair tile lies past M: nothing to publish, free the accumulator
                ptx::tc_fence_before();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive_cluster(acc_empty_addr[acc]);
                if ((acc ^= 1) == 0) acc_phase ^= 1;
                continue;
            }

            if (!LN && w.tail >= 0 && m0 < p.M) {
                // ---- K split of a last-wave tile: parts 1.. hand their accumulators over, part 0 collects them ----
                unsigned *flag = p.tail_flags + ((size_t)w.tail * 2 + rank) * 2 + h;
                const size_t slot = 32 * K2_EPI_THREADS;        // float4 per (tile, part, rank, half)
                if (w.part > 0) {
                    float4 *dst = p.tail_scratch + ((((size_t)w.tail * (p.tail_parts - 1) + (w.part - 1)) * 2 + rank) * 2 + h) * slot;
#pragma unroll 1
                    for (int c = 0; c < CHUNKS; ++c) {
                        uint32_t r[32];
                        ptx::tmem_ld_32x32(taddr + c * 32, r);
                        ptx::tmem_ld_wait();
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            dst[(c * 8 + i) * K2_EPI_THREADS + et] = make_float4(__uint_as_float(r[4 * i]), __uint_as_float(r[4 * i + 1]),
                                                                                 __uint_as_float(r[4 * i + 2]), __uint_as_float(r[4 * i + 3]));
                    }
                    epi_bar_sync(h);
                    if (et == 0) arrive_acq_rel(flag);      // its release covers the group's stores, ordered before it by the barrier
                    ptx::tc_fence_before();
                    __syncwarp();
                    if (lane == 0) { if (PAIR) ptx::mbar_arrive_cluster(acc_empty_addr[acc]); else ptx::mbar_arrive(&s.acc_empty[acc]); }
                    if ((acc ^= 1) == 0) acc_phase ^= 1;
                    continue;
                }
                if (et == 0 && !wait_counter<100>(flag, run * (unsigned)(p.tail_parts - 1), p.status, SITE_ARRIVAL, w.tail)) s.abort_flag = 1;
                epi_bar_sync(h);
                if (*(volatile int *)&s.abort_flag) { ok = false; break; }
#pragma unroll 1
                for (int c = 0; c < CHUNKS; ++c) {
                    uint32_t r[32];
                    ptx::tmem_ld_32x32(taddr + c * 32, r);
                    ptx::tmem_ld_wait();
                    for (int pp = 1; pp < p.tail_parts; ++pp) {
                        const float4 *src = p.tail_scratch + ((((size_t)w.tail * (p.tail_parts - 1) + (pp - 1)) * 2 + rank) * 2 + h) * slot;
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const float4 o = __ldcg(src + (c * 8 + i) * K2_EPI_THREADS + et);
                            r[4 * i] = __float_as_uint(__uint_as_float(r[4 * i]) + o.x);
                            r[4 * i + 1] = __float_as_uint(__uint_as_float(r[4 * i + 1]) + o.y);
                            r[4 * i + 2] = __float_as_uint(__uint_as_float(r[4 * i + 2]) + o.z);
                            r[4 * i + 3] = __float_as_uint(__uint_as_float(r[4 * i + 3]) + o.w);
                        }
                    }
                    ptx::tmem_st_32x32(taddr + c * 32, r);
                }
                ptx::tmem_st_wait();
            }

            if (LN) {
                // ---- sweep 1: activated values into registers, row statistics of this half tile ----
                float v[HALF];
                RowStat rs{0.f, 0.f, 0.f};
#pragma unroll
                for (int c = 0; c < CHUNKS; ++c) {
                    const int col0 = n0 + c * 32;
                    if (col0 < p.N) {
                        uint32_t r[32];
                        ptx::tmem_ld_32x32(taddr + c * 32, r);
                        ptx::tmem_ld_wait();
                        float (&x)[32] = reinterpret_cast<float (&)[32]>(v[c * 32]);      // this chunk's slice of the registers
#pragma unroll
                        for (int j = 0; j < 32; ++j) x[j] = __uint_as_float(r[j]) + sb[c * 32 + j];
                        apply_act_array<false>(p.e.act, x, p.e.scale);
                        rs = merge_stat(rs, chunk_moments(x, min(32, p.N - col0)));
                    }
                }
                // the accumulator is in registers: the TMEM buffer goes back to the MMA warp before the wait
                ptx::tc_fence_before();
                __syncwarp();
                if (lane == 0) { if (PAIR) ptx::mbar_arrive_cluster(acc_empty_addr[acc]); else ptx::mbar_arrive(&s.acc_empty[acc]); }
                float4 *stats = reinterpret_cast<float4 *>(p.partial);
                // Rows with more tiles than the grid has CTAs (pairs) cannot all be held on chip at once: every tile is
                // then computed twice.  Pass 0 publishes its triples and moves on (it never waits, so the grid always
                // gets through it); pass 1, which starts only when this unit has finished pass 0, recomputes the tile,
                // waits for the strip's triples (normally long there) and normalises.  Twice the arithmetic, and the
                // un-normalised tile still never leaves the SM.
                const bool publish = !p.two_pass || w.pass == 0, finish = !p.two_pass || w.pass == 1;
                if (publish && row < p.M) stats[(size_t)part * p.M + row] = make_float4(rs.n, rs.mean, rs.m2, 0.f);
                // ---- publish, then wait (bounded) for the other parts of this strip: one arrival per group by one
                //      thread (release: the group's triples, which the barrier orders before it; the acquiring polls
                //      and the next barrier make the other groups' triples readable past L1) ----
                epi_bar_sync(h);
                if (et == 0) {
                    if (publish) arrive_acq_rel(&p.counters[tm]);
                    if (finish && !wait_counter<0>(&p.counters[tm], run * (unsigned)parts, p.status, SITE_ARRIVAL, tm)) s.abort_flag = 1;
                }
                epi_bar_sync(h);
                if (*(volatile int *)&s.abort_flag) { ok = false; break; }
                if (!finish) {
                    if ((acc ^= 1) == 0) acc_phase ^= 1;
                    continue;
                }
                // the strip's parts combined in part order, all at once (same result on every CTA)
                float rstd = 0.f, shift = 0.f;
                if (row < p.M) shift = -combine_row_moments<false>(stats, parts, p.M, row, p.e.eps, rstd) * rstd;
                // ---- sweep 2: normalise the registers and store ----
                {
                    uint4 *patch = s.store_patch[warp - EPI_WARP0];
#pragma unroll
                    for (int c = 0; c < HALF / 32; ++c) {
                        uint4 w4[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            float y[8];
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                const int cc = c * 32 + i * 8 + j;
                                y[j] = fmaf(fmaf(v[cc], rstd, shift), sg[cc], sbe[cc]);
                            }
                            w4[i].x = ptx::pack16x2(y[0], y[1], p.f16);
                            w4[i].y = ptx::pack16x2(y[2], y[3], p.f16);
                            w4[i].z = ptx::pack16x2(y[4], y[5], p.f16);
                            w4[i].w = ptx::pack16x2(y[6], y[7], p.f16);
                        }
                        if (n0 + c * 32 < p.N)
                            k2_store_row_pieces(patch, lane, w4, reinterpret_cast<__nv_bfloat16 *>(p.out), m0 + 32 * q, p.M, p.N, n0 + c * 32);
                    }
                }
                if ((acc ^= 1) == 0) acc_phase ^= 1;
                continue;
            }

            // ---- plain epilogue and the row reductions: one sweep over the half tile (epilogue_tmem.cuh) ----
            const int tgt = (p.e.red == FORGE_RED_CROSS_ENTROPY && row < p.M) ? __ldg(reinterpret_cast<const int *>(p.gamma) + row) : -1;
            HalfTileRow mine;
            half_tile_sweep<false, CHUNKS>(taddr, n0, p.N, p.e, sb, sg, tgt,
                [&](int col0, const float (&v)[32], int) {
                    uint4 w4[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        w4[i].x = ptx::pack16x2(v[i * 8 + 0], v[i * 8 + 1], p.f16);
                        w4[i].y = ptx::pack16x2(v[i * 8 + 2], v[i * 8 + 3], p.f16);
                        w4[i].z = ptx::pack16x2(v[i * 8 + 4], v[i * 8 + 5], p.f16);
                        w4[i].w = ptx::pack16x2(v[i * 8 + 6], v[i * 8 + 7], p.f16);
                    }
                    k2_store_row_pieces(s.store_patch[warp - EPI_WARP0], lane, w4, reinterpret_cast<__nv_bfloat16 *>(p.out),
                                        m0 + 32 * q, p.M, p.N, col0);
                }, mine);
            // accumulator drained: hand the TMEM buffer back to the MMA warp
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) { if (PAIR) ptx::mbar_arrive_cluster(acc_empty_addr[acc]); else ptx::mbar_arrive(&s.acc_empty[acc]); }
            if (reduce || p.e.red == FORGE_RED_LOGSUMEXP || p.e.red == FORGE_RED_CROSS_ENTROPY)
                strip_fold<false>(p.e, mine, p.partial, part, parts, p.M, p.N, row, et == 0, &p.counters[tm], &s.last_flag[h],
                                  [h] { epi_bar_sync(h); }, reinterpret_cast<float *>(p.out), p.rowg, p.strips_done);
            if ((acc ^= 1) == 0) acc_phase ^= 1;
        }
    }

    // ---------------- mean chain: residual rows ----------------
    // Y[m, :] = X[m, :] + gelu(mean)[m] for all of Y ([M,K]) once every strip has published its
    // values, spread over the whole grid, 16 bytes per access (a strip written by the epilogue group
    // that finished it would stall that CTA's pipeline for the duration).  CTAs wait on one another
    // here: the launch is cooperative (all CTAs resident) and the wait is bounded.
    if (!LN && p.e.red == FORGE_RED_MEAN_GELU_RESIDUAL) {
        if (threadIdx.x == 0 && !wait_counter<200>(p.strips_done, run * (unsigned)p.tiles_m, p.status, SITE_ARRIVAL, (int)blockIdx.x))
            s.abort_flag = 1;
        __syncthreads();
        if (!*(volatile int *)&s.abort_flag) {
            const size_t k8 = (size_t)(p.K >> 3);
            const bool f16 = p.f16;
            residual_rows<8>(reinterpret_cast<const uint4 *>(p.X), reinterpret_cast<uint4 *>(p.out), k8, (size_t)p.M * k8,
                          (size_t)blockIdx.x * THREADS + threadIdx.x, (size_t)gridDim.x * THREADS,
                          [&](size_t row) { return __ldcg(p.rowg + row); },
                          [f16](uint4 &x, float g) {
                              uint32_t *w = reinterpret_cast<uint32_t *>(&x);
#pragma unroll
                              for (int i = 0; i < 4; ++i) {
                                  float lo, hi;
                                  ptx::unpack16x2(w[i], f16, lo, hi);
                                  w[i] = ptx::pack16x2(lo + g, hi + g, f16);
                              }
                          });
        } else {
            ok = false;
        }
    }

    // ---------------- teardown ----------------
    if (!ok) __nanosleep(200000);      // give-up path: let copies and MMAs already in flight land
    ptx::tc_fence_before();
    __syncthreads();
    if (PAIR) ptx::cluster_sync_all();     // the peer no longer reads this CTA's shared memory or signals its barriers
    if (warp == 1) {
        ptx::tc_fence_after();
        if (PAIR) ptx::tmem_dealloc_pair(tmem_base, K2_TMEM_COLS);
        else ptx::tmem_dealloc(tmem_base, K2_TMEM_COLS);
    }
    if (p.cooperative && threadIdx.x == 0) run_index_end(p.gen, run);
}

// ---- host side ---------------------------------------------------------------------------
// CTA pairs need at least two 128-row strips and two SMs (a tuning build with -DFORGE_K2_PAIR=0
// runs one CTA per tile throughout).
static bool k2_use_pair(const forge_fused_linear_desc_t &d, int sm_count)
{
    return FORGE_K2_PAIR != 0 && d.M > K2_BM && sm_count >= 2;
}

// Grid, K split of the last wave and workspace layout of the non-LayerNorm kernel (tile_schedule.cuh).
constexpr int K2_TAIL_MIN_KB = 16;        // a part is worth its hand-over only with 1024 k or more
struct K2Layout : ScheduleLayout {
    bool pair;
    int64_t grid;
};

static K2Layout k2_layout(const forge_fused_linear_desc_t &d, int sm_count)
{
    const bool pair = k2_use_pair(d, sm_count);
    const int64_t tiles_m = (d.M + K2_BM - 1) / K2_BM, tiles_n = (d.N + K2_BN - 1) / K2_BN;
    const bool lse = d.red == FORGE_RED_LOGSUMEXP || d.red == FORGE_RED_CROSS_ENTROPY;      // float4 partials
    const bool chain = d.red == FORGE_RED_MEAN_GELU_RESIDUAL;
    const bool fold = d.red == FORGE_RED_SUM || d.red == FORGE_RED_MAX || chain || lse;      // one partial per row and half tile
    K2Layout L = {};
    static_cast<ScheduleLayout &>(L) = schedule_layout(
        tiles_m, tiles_n, (pair ? (tiles_m + 1) / 2 : tiles_m) * tiles_n, pair ? sm_count / 2 : sm_count,
        (int)((d.K + K2_BK - 1) / K2_BK), FORGE_K2_TAIL_SPLIT != 0 && d.red != FORGE_RED_LAYERNORM, K2_TAIL_MIN_KB,
        fold ? (lse ? 4 : 1) * 2 * (size_t)tiles_n * (size_t)d.M : 0, chain, d.M);
    L.pair = pair;
    L.grid = pair ? 2 * L.ctas : L.ctas;
    return L;
}

forge_status_t k2_plan(const forge_fused_linear_desc_t &d, int sm_count, forge_plan_info_t *info, WorkspaceLayout *wl)
{
    if (d.M > 0x7fffffff || d.N > 0x7fffffff || d.K > 0x7fffffff) return FORGE_ERR_UNSUPPORTED;
    const K2Layout L = k2_layout(d, sm_count);
    if (L.tiles_m * L.tiles_n > 0x7fffffff) return FORGE_ERR_UNSUPPORTED;
    info->kernel = FORGE_KERNEL_BF16_TCGEN05;
    info->tile_m = L.pair ? 2 * K2_BM : K2_BM;
    info->tile_n = K2_BN;
    info->tile_k = K2_BK;
    info->stages = L.pair ? K2Ring<true>::STAGES : (d.M <= K2_BM / 2 ? K2_STAGES_SHORT : K2Ring<false>::STAGES);
    info->cluster = L.pair ? 2 : 1;
    info->threads = K2Shape<false>::THREADS;
    info->grid = L.grid;
    info->smem_bytes = (int64_t)K2_SMEM_BYTES;
    wl->partial_floats = L.partial_floats;
    wl->counters = L.counters;
    return FORGE_OK;
}

// CTAs wait on one another in the mean chain (all strips) and in the K split (part 0 on the others).
static bool k2_ctas_wait(const Handle &h) { return h.d.red == FORGE_RED_MEAN_GELU_RESIDUAL || k2_layout(h.d, h.sm_count).tail_parts > 1; }

template <bool LN, bool PAIR>
static forge_status_t k2_prepare()
{
    return cudaFuncSetAttribute(k2_bf16_tcgen05_kernel<LN, PAIR>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)K2_SMEM_BYTES) == cudaSuccess ? FORGE_OK : FORGE_ERR_CUDA;
}

// Kernels whose CTAs wait on one another (LayerNorm strips, the mean chain's residual phase) need the
// whole grid resident at once.
template <bool LN, bool PAIR>
static forge_status_t k2_check_residency(const Handle &h)
{
    int coop = 0, per_sm = 0;
    if (cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, h.d.device) != cudaSuccess || !coop) return FORGE_ERR_CUDA;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k2_bf16_tcgen05_kernel<LN, PAIR>, K2Shape<LN>::THREADS, K2_SMEM_BYTES) != cudaSuccess ||
        (int64_t)per_sm * h.sm_count < h.info.grid)
        return FORGE_ERR_CUDA;
    return FORGE_OK;
}

forge_status_t k2_setup(Handle &h)
{
    const bool pair = h.info.cluster == 2;
    if ((pair ? k2_prepare<false, true>() : k2_prepare<false, false>()) != FORGE_OK) return FORGE_ERR_CUDA;
    if (!k2_ctas_wait(h)) return FORGE_OK;
    return pair ? k2_check_residency<false, true>(h) : k2_check_residency<false, false>(h);
}

forge_status_t k4_plan(const forge_fused_linear_desc_t &d, int sm_count, forge_plan_info_t *info, WorkspaceLayout *wl)
{
    const forge_status_t st = k2_plan(d, sm_count, info, wl);
    if (st != FORGE_OK) return st;
    const int64_t tiles_m = (d.M + K2_BM - 1) / K2_BM, tiles_n = (d.N + K2_BN - 1) / K2_BN;
    // the tiles of a strip wait for one another: they must all be resident at once, or every tile is computed
    // twice (see K2Item::pass)
    info->kernel = FORGE_KERNEL_BF16_TCGEN05_LN;
    info->threads = K2Shape<true>::THREADS;
    wl->partial_floats = 4 * 2 * (size_t)tiles_n * (size_t)d.M;          // one float4 per row and half tile
    wl->counters = (size_t)tiles_m + 2;                                   // strips, then run index and finished-CTA count
    return FORGE_OK;
}

// setmaxnreg.inc waits until the registers it asks for are free: the shares must fit into what a CTA is
// launched with, or the kernel is never launched.
template <bool PAIR>
static bool k4_register_shares_fit()
{
    cudaFuncAttributes fa;
    return cudaFuncGetAttributes(&fa, k2_bf16_tcgen05_kernel<true, PAIR>) == cudaSuccess &&
           fa.numRegs * K2Shape<true>::THREADS >= K4_REGS_NEEDED;
}

forge_status_t k4_setup(Handle &h)
{
    const bool pair = h.info.cluster == 2;
    if (!(pair ? k4_register_shares_fit<true>() : k4_register_shares_fit<false>())) return FORGE_ERR_CUDA;
    if ((pair ? k2_prepare<true, true>() : k2_prepare<true, false>()) != FORGE_OK) return FORGE_ERR_CUDA;
    return pair ? k2_check_residency<true, true>(h) : k2_check_residency<true, false>(h);
}

template <bool LN, bool PAIR>
static forge_status_t k2_launch_t(const Handle &h, const K2Params &p, cudaStream_t stream)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)h.info.grid);
    cfg.blockDim = dim3(K2Shape<LN>::THREADS);
    cfg.dynamicSmemBytes = K2_SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    int n = 0;
    if (PAIR) {
        attr[n].id = cudaLaunchAttributeClusterDimension;
        attr[n].val.clusterDim.x = 2;
        attr[n].val.clusterDim.y = 1;
        attr[n].val.clusterDim.z = 1;
        ++n;
    }
    // CTAs that wait on one another: a cooperative launch guarantees that all of them are resident
    if (p.cooperative && cooperative_launch_enabled()) {
        attr[n].id = cudaLaunchAttributeCooperative;
        attr[n].val.cooperative = 1;
        ++n;
    }
    cfg.attrs = attr;
    cfg.numAttrs = n;
    return cudaLaunchKernelEx(&cfg, k2_bf16_tcgen05_kernel<LN, PAIR>, h.tmX, h.tmW, p) == cudaSuccess ? FORGE_OK : FORGE_ERR_CUDA;
}

static forge_status_t k24_launch(Handle &h, const RunArgs &a, bool ln)
{
    const forge_fused_linear_desc_t &d = h.d;
    const bool pair = h.info.cluster == 2;
    forge_status_t st;
    if (h.tmX_ptr != a.X) {
        const bool short_x = !pair && d.M <= K2_BM / 2;          // the box is what TMA writes: 64 rows, 8 KiB
        if ((st = encode_tmap_16(&h.tmX, a.X, (uint64_t)d.M, (uint64_t)d.K, short_x ? K2_BM / 2 : K2_BM, K2_BK, d.dtype == FORGE_F16)) != FORGE_OK) return st;
        h.tmX_ptr = a.X;
    }
    if (h.tmW_ptr != a.W) {
        if ((st = encode_tmap_16(&h.tmW, a.W, (uint64_t)d.N, (uint64_t)d.K, pair ? K2_BN / 2 : K2_BN, K2_BK, d.dtype == FORGE_F16)) != FORGE_OK) return st;
        h.tmW_ptr = a.W;
    }
    K2Params p = {};
    p.f16 = d.dtype == FORGE_F16;
    p.b = (const uint16_t *)a.b;
    p.X = (const uint16_t *)a.X;
    p.gamma = (const uint16_t *)a.gamma;
    p.beta = (const uint16_t *)a.beta;
    p.out = a.out;
    p.M = (int)d.M;
    p.N = (int)d.N;
    p.K = (int)d.K;
    p.e = Epilogue{(int)d.act, (int)d.red, d.scale, d.ln_eps, d.has_bias};
    p.partial = h.ws.partial;
    p.counters = h.ws.counters;
    p.status = h.ws.status;
    p.tiles_m = (int)((d.M + K2_BM - 1) / K2_BM);
    p.tiles_n = (int)((d.N + K2_BN - 1) / K2_BN);
    p.num_kb = (int)((d.K + K2_BK - 1) / K2_BK);
    p.short_x = !pair && d.M <= K2_BM / 2;
    p.ws_floats = h.ws.partial_floats;
    p.ws_counters = h.ws.counter_words;
    p.group_m = pair ? K2_GROUP_M / 2 : K2_GROUP_M;      // 4096 rows either way
    p.k_serpentine = FORGE_K2_K_SERPENTINE && k_serpentine_pays(d, h.info.grid / h.info.cluster, pair ? 2 * K2_BM : K2_BM, K2_BN, ln ? 0 : K2_GROUP_M * K2_BM, 2, h.l2_bytes);
    if (!ln) {
        const K2Layout L = k2_layout(d, h.sm_count);
        p.rowg = h.ws.partial + L.rowg_off;
        p.strips_done = h.ws.counters + L.strips_done_idx;
        p.tail_parts = L.tail_parts;
        p.tail_kb = L.tail_kb;
        p.tail_scratch = reinterpret_cast<float4 *>(h.ws.partial + L.scratch_off);
        p.tail_flags = h.ws.counters + L.tail_flags_idx;
        p.gen = h.ws.counters + L.gen_idx;
        p.cooperative = d.red == FORGE_RED_MEAN_GELU_RESIDUAL || L.tail_parts > 1;
        return pair ? k2_launch_t<false, true>(h, p, a.stream) : k2_launch_t<false, false>(h, p, a.stream);
    }
    p.tail_parts = 1;
    p.tail_kb = p.num_kb;
    p.cooperative = 1;
    p.gen = h.ws.counters + p.tiles_m;
    p.two_pass = p.tiles_n > h.info.grid / h.info.cluster;
    return pair ? k2_launch_t<true, true>(h, p, a.stream) : k2_launch_t<true, false>(h, p, a.stream);
}

forge_status_t k2_launch(Handle &h, const RunArgs &a) { return k24_launch(h, a, false); }
forge_status_t k4_launch(Handle &h, const RunArgs &a) { return k24_launch(h, a, true); }

}  // namespace forge
