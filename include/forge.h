/*
 * forge.h -- C interface of the B200 (sm_100a) fused linear operator
 *
 *     E = scale * act(X * W^T + b)            X [M,K], W [N,K], b [N]
 *     none:       Y[M,N]  = E
 *     sum / max:  out[M]  = sum_n E[m,n]  /  max_n E[m,n]
 *     layernorm:  Y[M,N]  = (E - mean_n E) / sqrt(var_n E + eps) * gamma[n] + beta[n]
 *     mean-gelu-residual: Y[M,K] = X + gelu_erf(mean_n (E - sub[n]))   (see forge_red_t)
 *     logsumexp / cross-entropy: out[M] = log sum_n exp E  [ - E[m, target[m]] ]
 *
 * The operation is the fused operator chain the paper's agents are asked to produce: one
 * kernel in place of a framework Linear (matmul + bias) followed by an element-wise
 * activation (Appendix A.1, "combining matmul + relu") and, optionally, a per-row statistic
 * computed from the accumulators without a trip through global memory (Appendix B.1, the
 * Linear + in-register epilogue proposal, whose stated difficulty is the aggregation across
 * output tiles).  Results are meant to agree with the unfused chain evaluated in double
 * precision within 1e-4 (fp32) -- the tolerance of Section 2.2 -- or 2e-2 (bf16 storage).
 *
 * Conventions for every entry point
 *   - No exceptions, no aborts: every failure is a forge_status_t return value.
 *   - All tensors are dense row-major with leading dimension K (X, W) or N (Y); the
 *     contraction runs over the contiguous axis of both X and W.
 *   - X, W, b, gamma, beta and Y share the descriptor's dtype; out[M] of sum/max is fp32.
 *   - Rounding of bf16 outputs is to nearest, ties to even.
 *   - There is no fallback: a descriptor the hand-written kernels cannot serve is rejected
 *     with FORGE_ERR_UNSUPPORTED, never computed some other way.
 */
#ifndef FORGE_H_
#define FORGE_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct forge_fused_linear_s *forge_fused_linear_t;   /* opaque handle */

typedef enum {
    FORGE_OK = 0,
    FORGE_ERR_INVALID_ARG = 1,   /* NULL pointer, bad enum, non-positive size, misalignment */
    FORGE_ERR_UNSUPPORTED = 2,   /* valid request that no kernel here serves              */
    FORGE_ERR_CUDA = 3,          /* a CUDA runtime/driver call failed (or no sm_100 GPU)  */
    FORGE_ERR_ALLOC = 4,         /* host or device allocation failed                      */
    FORGE_ERR_TIMEOUT = 5,       /* a bounded device-side wait gave up                    */
    FORGE_ERR_SCRATCH_LIMIT = 6, /* problem needs more scratch than the fixed buffer of   */
                                 /* forge_fused_linear_f32_reduce_static() holds          */
    FORGE_ERR_BOUNDS = 7         /* bounds-checked build only (-DFORGE_DEBUG_BOUNDS): a    */
                                 /* kernel computed an index outside its allocation; the  */
                                 /* access was skipped (last_status / last_wait_detail)   */
} forge_status_t;

typedef enum {
    FORGE_F32 = 0,               /* fp32 storage, fp32 FFMA arithmetic                    */
    FORGE_BF16 = 1,
    FORGE_F16 = 2,               /* IEEE half, same kernels as BF16                       */
    FORGE_F32_TF32X3 = 3
    /* fp32 storage (every tensor exactly as for FORGE_F32), contraction on the tensor cores:
     * each operand is split into a TF32 head and a TF32 tail and X W^T is accumulated in fp32
     * from the three products head*head, head*tail, tail*head (relative error of a product
     * about 2^-21), so the result stays within the 1e-4 of Section 2.2 with two orders of
     * magnitude to spare.  Needs K % 4 == 0, N % 4 == 0 and 16-byte aligned pointers.          */
} forge_dtype_t;

typedef enum {
    FORGE_ACT_IDENTITY = 0,
    FORGE_ACT_RELU = 1,          /* max(z, 0)                                            */
    FORGE_ACT_GELU_ERF = 2,      /* 0.5 z (1 + erf(z / sqrt 2))                          */
    FORGE_ACT_GELU_TANH = 3,     /* 0.5 z (1 + tanh(sqrt(2/pi) (z + 0.044715 z^3)))      */
    FORGE_ACT_SILU = 4           /* z / (1 + exp(-z))                                    */
} forge_act_t;

typedef enum {
    FORGE_RED_NONE = 0,
    FORGE_RED_SUM = 1,
    FORGE_RED_MAX = 2,
    FORGE_RED_LAYERNORM = 3,
    /* Population variance, eps inside the square root, gamma and beta applied after the
     * normalisation.  The N-tiles of a row strip exchange per-row (count, mean, M2) triples (the
     * "cross-tile aggregation" of Appendix B.1); the un-normalised values never leave the SM.
     * Any N: the tiles of a strip wait for one another, so when a strip has more tiles than the
     * grid has CTAs (pairs) -- N > 18944 on the tensor-core kernels, N > 37888 on the fp32 FFMA
     * kernel, on a B200 -- every tile is computed twice, once for the statistics and once to
     * normalise: twice the arithmetic, and still nothing un-normalised in global memory.         */
    FORGE_RED_MEAN_GELU_RESIDUAL = 4,
    /* The chain of the paper's Appendix B.1 case study (Linear, subtract, row mean, GELU,
     * residual add of the layer's input, all in one kernel):
     *     g[m] = gelu_erf(mean_n (E[m,n] - sub[n])),   Y[m,k] = X[m,k] + g[m]
     * The output is Y [M,K] (the shape of X) in dtype.  run() takes the subtract vector sub[N]
     * in its `gamma` argument (NULL: nothing is subtracted); `beta` is ignored.                */
    FORGE_RED_LOGSUMEXP = 5,
    /* out[m] = log sum_n exp(E[m,n]), fp32 [M]: the row statistic of a softmax over N, merged
     * across output tiles as (max, sum of exponentials) pairs; Y is never written (Section 4 of
     * the paper: warp-shuffle max / sum reductions of a cross-entropy kernel).                */
    FORGE_RED_CROSS_ENTROPY = 6
    /* out[m] = logsumexp_n E[m,:] - E[m, target[m]], fp32 [M]: the per-row loss of a classifier
     * head whose logits are never materialised.  run() takes the int32 class indices target[M]
     * (device pointer, each in [0, N)) in its `gamma` argument; `beta` is ignored.             */
} forge_red_t;

typedef struct {
    int64_t M, N, K;             /* all > 0                                              */
    forge_dtype_t dtype;         /* storage type of X, W, b, gamma, beta, Y              */
    forge_act_t act;
    forge_red_t red;
    float scale;                 /* multiplies act(...); 1.0f for none                   */
    float ln_eps;                /* FORGE_RED_LAYERNORM only                             */
    int has_bias;                /* 0: b is ignored and may be NULL                      */
    int device;                  /* CUDA device ordinal                                  */
} forge_fused_linear_desc_t;

/* Kernel families.  The choice is a pure function of the descriptor. */
typedef enum {
    FORGE_KERNEL_F32_FFMA = 1,        /* fp32 register-tiled FFMA GEMM, fused epilogue        */
    FORGE_KERNEL_BF16_TCGEN05 = 2,    /* bf16 TMA -> smem ring -> tcgen05.mma -> TMEM; CTA     */
                                      /* pairs (cta_group::2, 256x256 tiles) when M > 128      */
    FORGE_KERNEL_BF16_SKINNY = 3,     /* 16-bit, M <= 96: HBM-bound; rows of W are the M       */
                                      /* dimension of tcgen05.mma, X the N dimension (swap)    */
    FORGE_KERNEL_BF16_TCGEN05_LN = 4, /* bf16 tcgen05 whose epilogue merges row statistics    */
                                      /* across the N-tiles of a row strip (LayerNorm)         */
    FORGE_KERNEL_F32_TF32X3 = 5       /* fp32 operands split in shared memory into TF32 head   */
                                      /* and tail, three tcgen05.mma kind::tf32 per k-step     */
} forge_kernel_t;

typedef struct {
    forge_kernel_t kernel;
    int tile_m, tile_n, tile_k;  /* CTA tile (cluster tile when cluster > 1)              */
    int stages;                  /* depth of the shared-memory ring (0: not ring-based)   */
    int cluster;                 /* CTAs per cluster (1: no cluster)                      */
    int threads;                 /* threads per CTA                                       */
    int64_t grid;                /* CTAs launched, given sm_count                         */
    int64_t smem_bytes;          /* dynamic shared memory per CTA                         */
    int64_t workspace_bytes;     /* device scratch owned by the handle                    */
} forge_plan_info_t;

/*
 * Host-only: validate `desc` and report the kernel that create() would plan for a GPU with
 * `sm_count` multiprocessors.  Touches no device.  Returns FORGE_ERR_INVALID_ARG /
 * FORGE_ERR_UNSUPPORTED exactly as create() would for the same descriptor.
 * Kernel selection (Appendix B.1's point that the right fusion depends on whether the chain
 * is compute- or memory-bound): fp32 -> F32_FFMA; fp32 with TF32x3 arithmetic -> F32_TF32X3;
 * 16-bit with M <= 96 and neither LayerNorm nor the mean-GELU-residual chain -> BF16_SKINNY
 * (except a long K against few rows of W: K >= 24576 with N <= 16 x sm_count); 16-bit LayerNorm
 * -> BF16_TCGEN05_LN; other 16-bit -> BF16_TCGEN05.
 * Unsupported: 16-bit storage with K % 8 != 0 or N % 8 != 0 (16-byte row pitch); TF32x3 with
 * K % 4 != 0 or N % 4 != 0.
 */
forge_status_t forge_fused_linear_query_plan(const forge_fused_linear_desc_t *desc, int sm_count,
                                             forge_plan_info_t *info);

/*
 * Validate, plan, and allocate the handle's device workspace (per-tile partials, arrival
 * counters, a status word) on desc->device.  Host pointers: `desc` (read), `out` (written
 * with the new handle; NULL on failure).  Requires compute capability 10.x; otherwise
 * FORGE_ERR_CUDA.  Synchronous; launches no kernel on any user stream.
 */
forge_status_t forge_fused_linear_create(const forge_fused_linear_desc_t *desc, forge_fused_linear_t *out);

/*
 * Enqueue one evaluation on `cuda_stream` (a cudaStream_t; NULL = default stream).
 * DEVICE pointers, owned by the caller, 16-byte aligned, alive until the work completes:
 *   X [M,K], W [N,K], b [N] (may be NULL iff has_bias == 0), gamma, beta [N] (non-NULL iff
 *   layernorm), out: Y [M,N] in dtype (none, layernorm), fp32 [M] (sum, max, logsumexp,
 *   cross-entropy, whose int32 targets travel in `gamma`), or Y [M,K] in dtype
 *   (mean-gelu-residual, whose subtract vector travels in `gamma`).
 * Allocates nothing and does not synchronise.  Returns only argument / launch errors;
 * device-side give-ups are reported by forge_fused_linear_last_status().  At most one run
 * per handle may be in flight (the workspace belongs to the handle).  A call leaves nothing
 * on the host that a later call depends on (counters that CTAs wait on take their run index
 * from device memory), so a run captured into a CUDA graph can be replayed, also interleaved
 * with direct runs of the same handle.
 * Steps: operand fetch, contraction with fp32 accumulation, bias, activation, scale, row
 * reduction and store all happen inside the single kernel launched here (the fused form of
 * Appendix A.1 / B.1; nothing but the final result reaches global memory).
 */
forge_status_t forge_fused_linear_run(forge_fused_linear_t h, const void *X, const void *W, const void *b,
                                      const void *gamma, const void *beta, void *out, void *cuda_stream);

/*
 * Same operation with HOST buffers (pageable or pinned): copies the inputs to device
 * staging buffers owned by the handle (allocated on first use), runs, copies the result
 * back and synchronises.  Layouts and dtypes as for run(); bf16 data are raw 16-bit words.
 * A large X is walked in blocks of rows, each planned for its own row count, so a block's tiles may
 * accumulate over k in another order than run() on the whole problem: the results agree within
 * fp32 accumulation rounding (for 16-bit outputs: the last place), not necessarily bit for bit.
 */
forge_status_t forge_fused_linear_run_host(forge_fused_linear_t h, const void *X, const void *W, const void *b,
                                           const void *gamma, const void *beta, void *out);

/*
 * Read the handle's device status word.  Synchronises the device first.  FORGE_OK, or
 * FORGE_ERR_TIMEOUT if a bounded wait inside the last kernels expired (the output is then
 * undefined).  The word is cleared by this call.
 */
forge_status_t forge_fused_linear_last_status(forge_fused_linear_t h);

/*
 * Diagnostics of the give-up that the most recent last_status() call reported (host pointer
 * to 4 ints): [0] which wait (1 operand tile arrival, 2 ring stage release, 3 accumulator
 * ready, 4 accumulator release, 5 arrival of the other tiles of a row strip) or, for
 * FORGE_ERR_BOUNDS, which allocation (16 shared-memory ring, 17 tensor-memory columns,
 * 18 workspace partials, 19 workspace counters, 20 other shared memory), [1] a kernel-specific
 * detail word (FORGE_ERR_BOUNDS: the offending index), [2] CTA index, [3] thread index.  All
 * zero if none.
 */
forge_status_t forge_fused_linear_last_wait_detail(forge_fused_linear_t h, int detail[4]);

/*
 * Self-test of the bounded device-side wait that every kernel here uses (the paper's loop feeds
 * runtime failures back to its Judge, Section 2.2; a kernel that waits for ever gives no feedback
 * at all): runs a one-CTA kernel that waits on a barrier nothing signals, with a budget of
 * `budget_ms` (1..1000).  The expected return value is FORGE_ERR_TIMEOUT with detail[0] = 1 (the
 * operand-arrival wait), detail[1] = 0x5a5a, detail[2] = 0 (CTA), detail[3] = 32 (thread); the
 * kernel ends by itself and the device stays usable.  Synchronous; allocates and frees 256 bytes.
 */
forge_status_t forge_selftest_bounded_wait(int device, int budget_ms, int detail[4]);

/* Copy the plan chosen at create() into *info (host pointer). */
forge_status_t forge_fused_linear_get_plan(forge_fused_linear_t h, forge_plan_info_t *info);

/* Number of kernels run() launches per call for this handle (always >= 1). */
int forge_fused_linear_launches_per_run(forge_fused_linear_t h);

/* Name of the kernel family planned for this handle: forge_kernel_name() of its plan's kernel.
 * A static string; "no handle" for NULL. */
const char *forge_fused_linear_kernel_name(forge_fused_linear_t h);

/*
 * Measure the fp32 fused-multiply-add rate this device sustains: a kernel whose loop body is
 * nothing but independent register-to-register FMAs runs on every SM for about `milliseconds`
 * (1..2000).  Writes the rate in TFLOP/s (2 flop per FMA) to *tflops and, if the pointer is not
 * NULL, the SM clock that rate corresponds to at 128 FMA lanes per SM to *sm_mhz_effective (host
 * pointers).  This is the measured ceiling the fp32 FFMA kernel's throughput is compared with --
 * the paper's Judge reads pipe utilisation for the same purpose (Appendix C).  Synchronous;
 * allocates and frees 256 bytes.
 */
forge_status_t forge_selftest_ffma_rate(int device, int milliseconds, double *tflops, double *sm_mhz_effective);

/*
 * Measure what the memory system of this device delivers to a kernel that only reads: one thread per
 * SM keeps four 32-KiB bulk copies (global -> shared memory) in flight over a contiguous share of a
 * 256-MiB buffer, nothing is computed.  Three such buffers (768 MiB, allocated and freed here) are read in
 * turn, so nothing is served from L2.  Writes GB/s (1e9 bytes) of 30 launches issued back to back to
 * *gbs_back_to_back and, if the pointer is not NULL, of the median of 11 launches with a synchronise
 * after each to *gbs_single (host pointers).  This is the measured ceiling the HBM-bound skinny-M
 * kernel is compared with -- the paper's Judge reads `dram__throughput` for the same question
 * (Appendix C).  Synchronous.
 */
forge_status_t forge_selftest_read_stream(int device, double *gbs_back_to_back, double *gbs_single);

/*
 * Row sum / row max of the fp32 fused linear without a handle and without any allocation.
 * (The paper has no counterpart to this entry point: it exists for the benefit of callers,
 * not of the method.)
 *
 * Who needs it: code that may not call cudaMalloc when it wants the result -- a plugin
 * running inside someone else's memory pool or under a fixed memory budget, a real-time or
 * latency-critical loop where an allocation (which can synchronise the whole device) is not
 * acceptable, a process that has handed all device memory to its own allocator and cannot
 * get more from the driver.  create() cannot serve them: it allocates the workspace in which
 * the N-tiles of a row strip leave their partial sums / maxima and count their arrivals.
 *
 * Here that workspace is a fixed array of FORGE_STATIC_SCRATCH_BYTES inside the library
 * image; every GPU that loads the library carries it until the process ends.  The call
 * needs, for ceil(M/128) row strips and ceil(N/128) column tiles,
 *     roundup(4 * ceil(M/128), 256) + (ceil(N/128) > 1 ? 4 * M * ceil(N/128) : 0)  bytes;
 * a problem that needs more is refused with FORGE_ERR_SCRATCH_LIMIT (nothing is launched).
 *
 * Computes out[m] = sum_n or max_n of scale * act(X W^T + b), fp32, on the CURRENT device.
 * DEVICE pointers, 4-byte aligned (16-byte alignment of X and W with K % 4 == 0 enables the
 * 128-bit loads): X [M,K], W [N,K], b [N] or NULL for no bias, out [M] fp32.  `red` must be
 * FORGE_RED_SUM or FORGE_RED_MAX.  Asynchronous on `cuda_stream`; calls neither cudaMalloc
 * nor cudaFree nor any allocating library routine.
 *
 * The first call on each device looks up the device address of the array (a runtime query);
 * make that first call outside any stream capture.  All calls in the process share the one
 * array per device, and it keeps the previous call's contents: this function zeroes the
 * arrival counters on the stream before the kernel, but two calls whose kernels overlap on
 * the GPU (different streams, no dependency) race on it and give wrong results -- keep
 * calls on one device ordered.  Results agree with the handle-based path within fp32 rounding;
 * the tile shape may differ (this entry point always uses 128x128 tiles and walks all of K in
 * one CTA, a handle may plan 64x64 tiles with K slices), and they are bit-identical only when
 * the handle plans the same tiles.
 */
#define FORGE_STATIC_SCRATCH_BYTES (1u << 20)
forge_status_t forge_fused_linear_f32_reduce_static(int64_t M, int64_t N, int64_t K, forge_act_t act,
                                                    forge_red_t red, float scale, const void *X,
                                                    const void *W, const void *b, void *out,
                                                    void *cuda_stream);

/* Free the workspace, staging buffers and the handle.  NULL is FORGE_ERR_INVALID_ARG. */
forge_status_t forge_fused_linear_destroy(forge_fused_linear_t h);

/* Static strings; never NULL. */
const char *forge_status_string(forge_status_t s);
const char *forge_kernel_name(forge_kernel_t k);

#ifdef __cplusplus
}
#endif
#endif /* FORGE_H_ */
