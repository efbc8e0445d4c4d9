// K3: 16-bit fused linear for M <= 32 (HBM-bound: the weight matrix is read once and that is
// the whole cost).
//
// Each CTA owns a contiguous range of 8-column groups of the output (8 rows of W per group)
// sized so that all CTAs stream the same number of bytes.  A producer warp streams W (and
// the matching slice of X, which stays L2-resident) through a TMA ring (a stage is 128 k of
// every row of the strip: two boxes, so 256 contiguous bytes per row); 8 consumer warps feed
// the tiles to mma.sync.m16n8k16 straight from shared memory (ldmatrix on the
// 128-byte-swizzled layout).  X is the A operand: MT = 1 or 2 tiles of 16 rows (rows past
// M are TMA zero fill), every W fragment is used for all of them.  The warps split the work
// 4 (quarters of the strip's columns) x 2 (K: ring stages are dealt round-robin), so the
// partial accumulators of the 2 K-slices are summed -- before bias and activation, which are
// nonlinear -- through shared memory in a fixed order.  Row sum / max / softmax statistics:
// two shuffles inside the 4-lane groups that share a row, then per-CTA partials folded by the
// CTA that arrives last.
//
// Every thread of the CTA stays resident until the common exit barrier, so that no copy can
// still be in flight towards the shared memory of a CTA that has left.
#include "common.cuh"
#include "plan.h"
#include "sm100_ptx.cuh"

namespace forge {

constexpr int K3_BK = 64;                       // k per TMA box: one 128-byte swizzle row
constexpr int K3_KB = 2;                        // boxes per stage: 256 contiguous bytes of every W row at a time
constexpr int K3_MAX_GROUPS = 14;               // 8-column groups per strip (112 rows of W)
constexpr int K3_PAD_GROUPS = 16;               // group count the warp layout and the scratch arrays are sized for
constexpr int K3_MAX_STAGES = 6;
constexpr int K3_MAX_M = 32;                    // beyond this the mma.sync rate, not the weight stream, sets the time
constexpr int K3_KSPLIT = 2, K3_NSPLIT = 4;
constexpr int K3_CONSUMER_WARPS = K3_KSPLIT * K3_NSPLIT;
constexpr int K3_CONSUMERS = K3_CONSUMER_WARPS * 32;
constexpr int K3_THREADS = K3_CONSUMERS + 32;
constexpr uint32_t K3_WBOX_BYTES = K3_MAX_GROUPS * 8 * K3_BK * 2;  // 14 KiB: one W box of a full strip
constexpr uint32_t K3_W_BYTES = K3_KB * K3_WBOX_BYTES;
constexpr int K3_GH = K3_PAD_GROUPS / K3_NSPLIT;                   // groups per warp column part

// Ring geometry for MT row tiles of X: a stage is the W boxes plus MT 2-KiB X boxes per k block.
template <int MT> struct K3Ring {
    static constexpr uint32_t XBOX_BYTES = 16 * MT * K3_BK * 2;
    static constexpr uint32_t X_BYTES = K3_KB * XBOX_BYTES;
    static constexpr uint32_t STAGE_BYTES = K3_W_BYTES + X_BYTES;   // 32 / 36 KiB
    static constexpr int STAGES = MT == 1 ? 6 : 4;
    // A ring slot must be consumed by the same warps on every pass.  The phase-parity wait only
    // tells "one phase further" from "not yet"; a warp that never consumed pass n of a slot has
    // nothing that orders its wait for pass n+1 after the completion of pass n, and would read a
    // spurious success while pass n is still in flight.
    static_assert(STAGES % K3_KSPLIT == 0, "each ring slot belongs to one K-slice");
    static_assert(STAGES <= K3_MAX_STAGES, "barrier arrays");
};
constexpr size_t K3_RING_BYTES = (size_t)K3Ring<1>::STAGES * K3Ring<1>::STAGE_BYTES;     // 192 KiB, the largest
static_assert((size_t)K3Ring<2>::STAGES * K3Ring<2>::STAGE_BYTES <= K3_RING_BYTES, "ring");

struct K3Smem {
    uint64_t full[K3_MAX_STAGES];
    uint64_t empty[K3_MAX_STAGES];
    float4 red[K3_KSPLIT][K3_PAD_GROUPS][32];    // partial accumulators of the K-slices, one 16-row tile at a time
    float rowred[K3_PAD_GROUPS * 16];            // per (group, row) or per (chunk, row) row statistics
    float rowred_s[K3_PAD_GROUPS * 16];          // softmax statistics: sum of exponentials ...
    float rowred_t[K3_PAD_GROUPS * 16];          // ... and the target's logit
    int last_flag;
    int abort_flag;
};
constexpr size_t K3_SMEM_BYTES = 1024 + K3_RING_BYTES + sizeof(K3Smem);

struct K3Params {
    int f16;              // IEEE half (1) or bfloat16 (0) storage
    const uint16_t *b;
    const int *target;    // cross-entropy: class index per row
    void *out;
    int M, N, K;
    Epilogue e;
    float *partial;       // [grid][16 MT] floats, or float4 (softmax statistics)
    unsigned *counters;   // [1]
    int *status;
    int num_kb;
    int groups;           // N / 8
    int box_groups;       // groups per strip = rows of the W box / 8
    long long ws_floats;  // extent of `partial` (bounds-checked build)
};

__device__ __forceinline__ void k3_consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(K3_CONSUMERS) : "memory"); }

template <bool F16, int MT>
__global__ void __launch_bounds__(K3_THREADS, 1)
k3_bf16_skinny_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW, const K3Params p)
{
    using Ring = K3Ring<MT>;
    constexpr int STAGES = Ring::STAGES;
    constexpr uint32_t STAGE_BYTES = Ring::STAGE_BYTES, XBOX_BYTES = Ring::XBOX_BYTES;
    constexpr int ROWS = 16 * MT;                // rows of the output this kernel carries
    extern __shared__ uint8_t smem_raw[];
    uint8_t *ring = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    K3Smem &s = *reinterpret_cast<K3Smem *>(ring + K3_RING_BYTES);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // this CTA's share of the column groups, and its strips
    const int g_lo = (int)((long long)p.groups * blockIdx.x / gridDim.x);
    const int g_hi = (int)((long long)p.groups * (blockIdx.x + 1) / gridDim.x);
    const int strips = (g_hi - g_lo + p.box_groups - 1) / p.box_groups;
    const uint32_t wbox_bytes = (uint32_t)p.box_groups * 8 * K3_BK * 2;       // multiple of 1024
    const uint32_t stage_tx = K3_KB * wbox_bytes + Ring::X_BYTES;

    if (threadIdx.x == 0) {
        for (int i = 0; i < STAGES; ++i) { ptx::mbar_init(&s.full[i], 1); ptx::mbar_init(&s.empty[i], K3_NSPLIT); }
        s.abort_flag = 0;
        s.last_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tmap(&tmX);
        ptx::prefetch_tmap(&tmW);
    }
    // This kernel is short (tens of microseconds), so the gap between two launches matters: let
    // the next launch set itself up on each SM as soon as this CTA leaves it, and touch global
    // memory only once everything earlier in the stream has completed.
    ptx::pdl_launch_dependents();
    __syncthreads();
    ptx::pdl_wait();

    if (warp == K3_CONSUMER_WARPS) {
        // ---------------- TMA producer ----------------
        if (ptx::elect_one()) {
            int slot = 0;
            uint32_t phase = 0;
            bool ok = true;
            const int kb_rot = (int)((long long)p.num_kb * blockIdx.x / gridDim.x);
            for (int st = 0; st < strips && ok; ++st) {
                const int row0 = (g_lo + st * p.box_groups) * 8;
                for (int i = 0; i < p.num_kb; ++i) {
                    // CTAs start at different k: if all of them walked K in lock step, the requests in
                    // flight would share their low address bits and pile onto a few DRAM channels
                    int kb = i + kb_rot;
                    if (kb >= p.num_kb) kb -= p.num_kb;
                    if (!ptx::mbar_wait(&s.empty[slot], phase ^ 1, p.status, SITE_STAGE_EMPTY, (slot << 16) | (kb & 0xffff))) { ok = false; break; }
                    if (!in_bounds(p.status, BOUNDS_RING, (long long)slot * STAGE_BYTES, STAGE_BYTES, (long long)K3_RING_BYTES)) { ok = false; break; }
                    uint8_t *dst = ring + (size_t)slot * STAGE_BYTES;
                    ptx::mbar_expect_tx(&s.full[slot], stage_tx);
                    // a box that starts at or past K (ragged last stage) is all zero fill
#pragma unroll
                    for (int j = 0; j < K3_KB; ++j) {
                        ptx::tma_load_2d(dst + j * wbox_bytes, &tmW, &s.full[slot], (kb * K3_KB + j) * K3_BK, row0);
                        ptx::tma_load_2d(dst + K3_W_BYTES + j * XBOX_BYTES, &tmX, &s.full[slot], (kb * K3_KB + j) * K3_BK, 0);
                    }
                    if (++slot == STAGES) { slot = 0; phase ^= 1; }
                }
            }
            if (!ok) s.abort_flag = 1;
        }
    } else {
        // ---------------- consumers ----------------
        const int nh = warp % K3_NSPLIT;    // which part of the strip's groups
        const int ks = warp / K3_NSPLIT;    // which K-slice (ring stages with index % K3_KSPLIT == ks)
        const int t = threadIdx.x;          // 0..255
        const bool reduce = p.e.red == FORGE_RED_SUM || p.e.red == FORGE_RED_MAX;
        const bool softmax = p.e.red == FORGE_RED_LOGSUMEXP || p.e.red == FORGE_RED_CROSS_ENTROPY;
        bool ok = true;
        // threads 0..15 carry row (16 mt + t) of the output across groups and strips
        float running[MT], running_s[MT], running_t[MT];      // sum or max (softmax: max, sum exp, target logit)
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
            running[mt] = p.e.red == FORGE_RED_SUM ? 0.f : -INFINITY;
            running_s[mt] = running_t[mt] = 0.f;
        }

        // ldmatrix lane addressing on the 128-byte-swizzled tiles (16-byte chunk c of row r
        // sits at r*128 + ((c ^ (r & 7)) << 4)).
        const int lm = lane >> 3, lr = lane & 7;
        const int a_row = (lm & 1) * 8 + lr, a_chunk = lm >> 1;     // X: (r0-7,k0-7) (r8-15,k0-7) (r0-7,k8-15) (r8-15,k8-15)
        const int b_row = (lm >> 1) * 8 + lr, b_chunk = lm & 1;     // W: (g,k0-7) (g,k8-15) (g+1,k0-7) (g+1,k8-15)

        // ring position of the next stage this warp consumes: sequence index, slot and phase
        int seq = ks, slot = ks;
        uint32_t phase = 0;
        int seq_end = 0;                    // first sequence index past the current strip

        for (int st = 0; st < strips; ++st) {
            seq_end += p.num_kb;
            const int gbase = g_lo + st * p.box_groups;
            const int ng = min(p.box_groups, p.groups - gbase);      // groups present in this strip's box
            float acc[MT][K3_GH][4];
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                for (int g = 0; g < K3_GH; ++g) acc[mt][g][0] = acc[mt][g][1] = acc[mt][g][2] = acc[mt][g][3] = 0.f;

            for (; seq < seq_end; seq += K3_KSPLIT) {
                if (ok && !ptx::mbar_wait(&s.full[slot], phase, p.status, SITE_TMA_FULL, (slot << 16) | (seq & 0xffff))) ok = false;
                if (ok && !in_bounds(p.status, BOUNDS_RING, (long long)slot * STAGE_BYTES, STAGE_BYTES, (long long)K3_RING_BYTES)) ok = false;
                if (ok) {
                    const uint32_t wbase = ptx::smem_u32(ring + (size_t)slot * STAGE_BYTES);
                    const uint32_t xbase = wbase + K3_W_BYTES;
#pragma unroll
                    for (int kq = 0; kq < K3_KB * K3_BK / 16; ++kq) {
                        const int j = kq / (K3_BK / 16), kk = kq % (K3_BK / 16);     // box, 16-wide step inside it
                        uint32_t a[MT][4];
#pragma unroll
                        for (int mt = 0; mt < MT; ++mt)      // (16 mt + a_row) & 7 == a_row & 7: same swizzle phase
                            ptx::ldmatrix_x4(a[mt], xbase + j * XBOX_BYTES + (mt * 16 + a_row) * 128 + (((2 * kk + a_chunk) ^ (a_row & 7)) << 4));
#pragma unroll
                        for (int gp = 0; gp < K3_GH / 2; ++gp) {
                            const int g0 = nh * K3_GH + gp * 2;
                            if (g0 < ng) {
                                uint32_t b[4];
                                const int r = g0 * 8 + b_row;
                                ptx::ldmatrix_x4(b, wbase + j * wbox_bytes + r * 128 + (((2 * kk + b_chunk) ^ (r & 7)) << 4));
#pragma unroll
                                for (int mt = 0; mt < MT; ++mt) {
                                    if (F16) {
                                        ptx::mma_m16n8k16_f16(acc[mt][gp * 2], a[mt], b[0], b[1]);
                                        ptx::mma_m16n8k16_f16(acc[mt][gp * 2 + 1], a[mt], b[2], b[3]);
                                    } else {
                                        ptx::mma_m16n8k16_bf16(acc[mt][gp * 2], a[mt], b[0], b[1]);
                                        ptx::mma_m16n8k16_bf16(acc[mt][gp * 2 + 1], a[mt], b[2], b[3]);
                                    }
                                }
                            }
                        }
                    }
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive(&s.empty[slot]);
                }
                slot += K3_KSPLIT;
                if (slot >= STAGES) { slot -= STAGES; phase ^= 1; }
            }

            // ---- per 16-row tile: sum the K-slices (fixed order), then the epilogue on the full
            //      pre-activations
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
#pragma unroll
                for (int g = 0; g < K3_GH; ++g)
                    s.red[ks][nh * K3_GH + g][lane] = make_float4(acc[mt][g][0], acc[mt][g][1], acc[mt][g][2], acc[mt][g][3]);
                k3_consumer_sync();

                const int r0 = mt * 16 + (lane >> 2), r1 = r0 + 8;          // output rows of this thread's fragment
                int tgt0 = -1, tgt1 = -1;
                if (p.e.red == FORGE_RED_CROSS_ENTROPY) {
                    if (r0 < p.M) tgt0 = __ldg(p.target + r0);
                    if (r1 < p.M) tgt1 = __ldg(p.target + r1);
                }
#pragma unroll
                for (int j = 0; j < K3_PAD_GROUPS * 32 / K3_CONSUMERS; ++j) {
                    const int g = warp + j * K3_CONSUMER_WARPS;        // fragment lane == this thread's lane
                    float4 z = s.red[0][g][lane];
#pragma unroll
                    for (int k = 1; k < K3_KSPLIT; ++k) {
                        const float4 o = s.red[k][g][lane];
                        z.x += o.x; z.y += o.y; z.z += o.z; z.w += o.w;
                    }
                    const int col = (gbase + g) * 8 + (lane & 3) * 2;
                    const bool live = g < ng && gbase + g < g_hi && col + 1 < p.N;   // in the box, in this CTA's share
                    float b0 = 0.f, b1 = 0.f;
                    if (live && p.e.has_bias) ptx::unpack16x2(__ldg(reinterpret_cast<const uint32_t *>(p.b + col)), F16, b0, b1);
                    float v[4] = {z.x + b0, z.y + b1, z.z + b0, z.w + b1};
                    apply_act_array<false>(p.e.act, v, p.e.scale);
                    const int q0 = g * 16 + (lane >> 2), q1 = q0 + 8;          // (group, row-in-tile) slots
                    if (reduce) {
                        float m0, m1;
                        if (p.e.red == FORGE_RED_SUM) {
                            m0 = live ? v[0] + v[1] : 0.f;
                            m1 = live ? v[2] + v[3] : 0.f;
                            m0 += __shfl_xor_sync(0xffffffffu, m0, 1);
                            m1 += __shfl_xor_sync(0xffffffffu, m1, 1);
                            m0 += __shfl_xor_sync(0xffffffffu, m0, 2);
                            m1 += __shfl_xor_sync(0xffffffffu, m1, 2);
                        } else {
                            m0 = live ? fmaxf(v[0], v[1]) : -INFINITY;
                            m1 = live ? fmaxf(v[2], v[3]) : -INFINITY;
                            m0 = fmaxf(m0, __shfl_xor_sync(0xffffffffu, m0, 1));
                            m1 = fmaxf(m1, __shfl_xor_sync(0xffffffffu, m1, 1));
                            m0 = fmaxf(m0, __shfl_xor_sync(0xffffffffu, m0, 2));
                            m1 = fmaxf(m1, __shfl_xor_sync(0xffffffffu, m1, 2));
                        }
                        if ((lane & 3) == 0) {
                            s.rowred[q0] = m0;
                            s.rowred[q1] = m1;
                        }
                    } else if (softmax) {
                        // (max, sum exp) of this thread's two columns of rows r0 and r1, merged over the
                        // four lanes that share the rows; the target's logit rides along
                        float m0 = live ? fmaxf(v[0], v[1]) : -INFINITY, m1 = live ? fmaxf(v[2], v[3]) : -INFINITY;
                        float s0 = live ? __expf(v[0] - m0) + __expf(v[1] - m0) : 0.f;
                        float s1 = live ? __expf(v[2] - m1) + __expf(v[3] - m1) : 0.f;
                        float t0 = 0.f, t1 = 0.f;
                        if (live) {
                            t0 = col == tgt0 ? v[0] : (col + 1 == tgt0 ? v[1] : 0.f);
                            t1 = col == tgt1 ? v[2] : (col + 1 == tgt1 ? v[3] : 0.f);
                        }
#pragma unroll
                        for (int sh = 1; sh <= 2; sh <<= 1) {
                            lse_merge<false>(m0, s0, __shfl_xor_sync(0xffffffffu, m0, sh), __shfl_xor_sync(0xffffffffu, s0, sh));
                            lse_merge<false>(m1, s1, __shfl_xor_sync(0xffffffffu, m1, sh), __shfl_xor_sync(0xffffffffu, s1, sh));
                            t0 += __shfl_xor_sync(0xffffffffu, t0, sh);
                            t1 += __shfl_xor_sync(0xffffffffu, t1, sh);
                        }
                        if ((lane & 3) == 0) {
                            s.rowred[q0] = m0; s.rowred_s[q0] = s0; s.rowred_t[q0] = t0;
                            s.rowred[q1] = m1; s.rowred_s[q1] = s1; s.rowred_t[q1] = t1;
                        }
                    } else if (live) {
                        uint16_t *Y = reinterpret_cast<uint16_t *>(p.out);
                        if (r0 < p.M) *reinterpret_cast<uint32_t *>(Y + (size_t)r0 * p.N + col) = ptx::pack16x2(v[0], v[1], F16);
                        if (r1 < p.M) *reinterpret_cast<uint32_t *>(Y + (size_t)r1 * p.N + col) = ptx::pack16x2(v[2], v[3], F16);
                    }
                }
                k3_consumer_sync();
                if (reduce && t < 16) {
                    for (int g = 0; g < K3_PAD_GROUPS; ++g) {
                        const float o = s.rowred[g * 16 + t];
                        running[mt] = p.e.red == FORGE_RED_SUM ? running[mt] + o : fmaxf(running[mt], o);
                    }
                }
                if (softmax && t < 16) {
                    for (int g = 0; g < K3_PAD_GROUPS; ++g) {
                        lse_merge<false>(running[mt], running_s[mt], s.rowred[g * 16 + t], s.rowred_s[g * 16 + t]);
                        running_t[mt] += s.rowred_t[g * 16 + t];
                    }
                }
            }
        }
        if (!ok) s.abort_flag = 1;

        // ---- fold the CTAs' partials: the last CTA to arrive does it, in a fixed order.  The ROWS
        //      rows are spread over the 256 threads as (row, chunk of CTAs); chunk results meet in
        //      shared memory ----
        if (reduce || softmax) {
            float *out = reinterpret_cast<float *>(p.out);
            float4 *part4 = reinterpret_cast<float4 *>(p.partial);
            if (gridDim.x == 1) {
                if (t < 16) {
#pragma unroll
                    for (int mt = 0; mt < MT; ++mt)
                        if (mt * 16 + t < p.M)
                            out[mt * 16 + t] = softmax ? running[mt] + __logf(running_s[mt]) - running_t[mt] : running[mt];
                }
            } else {
                if (t < 16) {
#pragma unroll
                    for (int mt = 0; mt < MT; ++mt) {
                        const size_t slot_i = (size_t)blockIdx.x * ROWS + mt * 16 + t;
                        if (!in_bounds(p.status, BOUNDS_PARTIAL, (long long)slot_i * (softmax ? 4 : 1), softmax ? 4 : 1, p.ws_floats)) continue;
                        if (softmax) part4[slot_i] = make_float4(running[mt], running_s[mt], running_t[mt], 0.f);
                        else p.partial[slot_i] = running[mt];
                    }
                }
                // one arrival per CTA, by one thread: its release covers the partials the barrier has ordered before
                // it, its acquire (and the next barrier) the other CTAs' partials read below.  No fence per thread: a
                // sequentially consistent fence on an SM with copies in flight costs microseconds.
                k3_consumer_sync();
                if (t == 0) s.last_flag = (arrive_acq_rel(&p.counters[0]) == gridDim.x - 1);
                k3_consumer_sync();
                if (s.last_flag) {
                    constexpr int CHUNKS = K3_CONSUMERS / ROWS;            // 16 or 8 chunks of CTAs per row
                    const int row = t % ROWS, chunk = t / ROWS;
                    float mx = p.e.red == FORGE_RED_SUM ? 0.f : -INFINITY, se = 0.f, tl = 0.f;
                    for (unsigned c = chunk; c < gridDim.x; c += CHUNKS) {
                        if (softmax) {
                            const float4 f = __ldcg(&part4[(size_t)c * ROWS + row]);
                            lse_merge<false>(mx, se, f.x, f.y);
                            tl += f.z;
                        } else {
                            const float o = __ldcg(&p.partial[(size_t)c * ROWS + row]);
                            mx = p.e.red == FORGE_RED_SUM ? mx + o : fmaxf(mx, o);
                        }
                    }
                    s.rowred[chunk * ROWS + row] = mx;
                    s.rowred_s[chunk * ROWS + row] = se;
                    s.rowred_t[chunk * ROWS + row] = tl;
                    k3_consumer_sync();
                    if (t < ROWS && t < p.M) {
                        mx = s.rowred[t]; se = s.rowred_s[t]; tl = s.rowred_t[t];
                        for (int j = 1; j < CHUNKS; ++j) {
                            if (softmax) {
                                lse_merge<false>(mx, se, s.rowred[j * ROWS + t], s.rowred_s[j * ROWS + t]);
                                tl += s.rowred_t[j * ROWS + t];
                            } else {
                                const float o = s.rowred[j * ROWS + t];
                                mx = p.e.red == FORGE_RED_SUM ? mx + o : fmaxf(mx, o);
                            }
                        }
                        out[t] = softmax ? mx + __logf(se) - tl : mx;
                    }
                    if (t == 0) p.counters[0] = 0u;
                }
            }
        }
    }

    // ---------------- common exit ----------------
    __syncthreads();
    // give-up path only: copies already issued may still be landing in this CTA's shared memory
    if (*(volatile int *)&s.abort_flag) __nanosleep(500000);
}

// ---- host side ---------------------------------------------------------------------------
static int k3_grid(const forge_fused_linear_desc_t &d, int sm_count)
{
    const int64_t groups = d.N / 8;
    return (int)(groups < sm_count ? groups : sm_count);
}
static int k3_box_groups(const forge_fused_linear_desc_t &d, int grid)
{
    const int64_t groups = d.N / 8;
    const int64_t per_cta = (groups + grid - 1) / grid;
    return (int)(per_cta < K3_MAX_GROUPS ? per_cta : K3_MAX_GROUPS);
}
static int k3_row_tiles(const forge_fused_linear_desc_t &d) { return d.M <= 16 ? 1 : 2; }

forge_status_t k3_plan(const forge_fused_linear_desc_t &d, int sm_count, forge_plan_info_t *info, WorkspaceLayout *wl)
{
    if (d.M > K3_MAX_M || d.N > 0x7fffffff || d.K > 0x7fffffff) return FORGE_ERR_UNSUPPORTED;
    if (d.red == FORGE_RED_LAYERNORM || d.red == FORGE_RED_MEAN_GELU_RESIDUAL) return FORGE_ERR_UNSUPPORTED;
    const int grid = k3_grid(d, sm_count), mt = k3_row_tiles(d);
    info->kernel = FORGE_KERNEL_BF16_SKINNY;
    info->tile_m = 16 * mt;
    info->tile_n = k3_box_groups(d, grid) * 8;
    info->tile_k = K3_KB * K3_BK;
    info->stages = mt == 1 ? K3Ring<1>::STAGES : K3Ring<2>::STAGES;
    info->cluster = 1;
    info->threads = K3_THREADS;
    info->grid = grid;
    info->smem_bytes = (int64_t)K3_SMEM_BYTES;
    const bool softmax = d.red == FORGE_RED_LOGSUMEXP || d.red == FORGE_RED_CROSS_ENTROPY;     // float4 partials
    const bool partials = (d.red == FORGE_RED_SUM || d.red == FORGE_RED_MAX || softmax) && grid > 1;
    wl->partial_floats = partials ? (size_t)grid * 16 * mt * (softmax ? 4 : 1) : 0;
    wl->counters = partials ? 1 : 0;
    return FORGE_OK;
}

template <bool F16, int MT>
static cudaError_t k3_prepare()
{
    return cudaFuncSetAttribute(k3_bf16_skinny_kernel<F16, MT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)K3_SMEM_BYTES);
}

forge_status_t k3_setup(Handle &)
{
    const bool ok = k3_prepare<false, 1>() == cudaSuccess && k3_prepare<false, 2>() == cudaSuccess &&
                    k3_prepare<true, 1>() == cudaSuccess && k3_prepare<true, 2>() == cudaSuccess;
    return ok ? FORGE_OK : FORGE_ERR_CUDA;
}

forge_status_t k3_launch(Handle &h, const RunArgs &a)
{
    const forge_fused_linear_desc_t &d = h.d;
    const int mt = h.info.tile_m / 16;
    forge_status_t st;
    if (h.tmX_ptr != a.X) {
        if ((st = encode_tmap_16(&h.tmX, a.X, (uint64_t)d.M, (uint64_t)d.K, 16 * mt, K3_BK, d.dtype == FORGE_F16)) != FORGE_OK) return st;
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
    p.num_kb = (int)((d.K + K3_KB * K3_BK - 1) / (K3_KB * K3_BK));
    p.groups = (int)(d.N / 8);
    p.box_groups = h.info.tile_n / 8;
    p.ws_floats = h.ws.partial_floats;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)h.info.grid);
    cfg.blockDim = dim3(K3_THREADS);
    cfg.dynamicSmemBytes = K3_SMEM_BYTES;
    cfg.stream = a.stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e;
#define K3_GO(F, T) e = cudaLaunchKernelEx(&cfg, k3_bf16_skinny_kernel<F, T>, h.tmX, h.tmW, p)
    if (p.f16) { if (mt == 1) K3_GO(true, 1); else K3_GO(true, 2); }
    else { if (mt == 1) K3_GO(false, 1); else K3_GO(false, 2); }
#undef K3_GO
    return e == cudaSuccess ? FORGE_OK : FORGE_ERR_CUDA;
}

}  // namespace forge
