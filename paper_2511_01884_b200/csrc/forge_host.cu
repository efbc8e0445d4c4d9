// The C interface: descriptor validation, kernel selection, workspace, launches.
#include <cstdlib>
#include <cstring>
#include <initializer_list>
#include <new>

#include "common.cuh"
#include "plan.h"
#include "sm100_ptx.cuh"

namespace forge {

namespace {

constexpr size_t kStatusBytes = 256;     // status word lives alone in the first 256 bytes

bool desc_enums_ok(const forge_fused_linear_desc_t &d)
{
    return (d.dtype == FORGE_F32 || d.dtype == FORGE_BF16 || d.dtype == FORGE_F16 || d.dtype == FORGE_F32_TF32X3) && d.act >= FORGE_ACT_IDENTITY &&
           d.act <= FORGE_ACT_SILU && d.red >= FORGE_RED_NONE && d.red <= FORGE_RED_CROSS_ENTROPY;
}

// Largest M served by the skinny kernel.  These problems are bound by the stream of W, and the skinny kernel
// spreads W over all SMs in equal shares, whatever N; the tile kernel has N/256 tiles to hand out.  As M grows the
// skinny kernel re-reads X from L2 once per 112-128 rows of W (the tile kernel once per 256), and past about 96 rows
// the tile kernel is level or ahead (measured on 16384 x 8192 and 32768 x 8192 weights, rotating copies:
// M = 96: 58 / 97 us against 66 / 104; M = 128: 63 / 113 against 67 / 105).  A tuning build may move the limit
// (-DFORGE_SKINNY_MAX_M=0..128) to compare the two kernels on the same problem.
#ifndef FORGE_SKINNY_MAX_M
#define FORGE_SKINNY_MAX_M 96
#endif
static_assert(FORGE_SKINNY_MAX_M >= 0 && FORGE_SKINNY_MAX_M <= 128, "the skinny kernel carries at most 128 rows");
constexpr int64_t skinny_max_m() { return FORGE_SKINNY_MAX_M; }
// One more case goes to the tile kernel: a long K against so few rows of W that an SM's share is 16 rows or fewer
// (N <= 16 x SMs).  The skinny kernel gives every CTA all of K for its rows, and 16 rows are too few bytes in flight
// per SM however the ring is cut; the tile kernel cuts K over the CTAs instead (measured, M = 16: 1024 x 65536
// 114 against 67 us, 2048 x 32768 61 against 52; but 2368 x 8192 21 against 35, 4096 x 16384 35 against 48).
bool skinny_serves(const forge_fused_linear_desc_t &d, int sm_count)
{
    if (d.M > skinny_max_m() || d.red == FORGE_RED_MEAN_GELU_RESIDUAL) return false;
    const int64_t groups = d.N / 8, ctas = groups < sm_count ? groups : sm_count;
    const int64_t rows_per_cta = ctas > 0 ? (groups + ctas - 1) / ctas * 8 : 0;
    return !(rows_per_cta <= 16 && d.K >= 24576);
}

forge_status_t plan_for(const forge_fused_linear_desc_t &d, int sm_count, forge_plan_info_t *info, WorkspaceLayout *wl)
{
    if (d.M <= 0 || d.N <= 0 || d.K <= 0 || !desc_enums_ok(d) || d.device < 0 || sm_count <= 0)
        return FORGE_ERR_INVALID_ARG;
    if (!(d.scale == d.scale) || !(d.ln_eps == d.ln_eps)) return FORGE_ERR_INVALID_ARG;   // NaN
    if (d.red == FORGE_RED_LAYERNORM && d.ln_eps < 0.f) return FORGE_ERR_INVALID_ARG;
    std::memset(info, 0, sizeof(*info));
    forge_status_t st;
    if (d.dtype == FORGE_F32) {
        st = k1_plan(d, sm_count, info, wl);
    } else if (d.dtype == FORGE_F32_TF32X3) {
        st = k5_plan(d, sm_count, info, wl);
    } else {
        if (d.K % 8 != 0 || d.N % 8 != 0) return FORGE_ERR_UNSUPPORTED;     // 16-byte row pitch for TMA
        if (d.red == FORGE_RED_LAYERNORM) st = k4_plan(d, sm_count, info, wl);
        else if (skinny_serves(d, sm_count)) st = k3_plan(d, sm_count, info, wl);
        else st = k2_plan(d, sm_count, info, wl);
    }
    if (st != FORGE_OK) return st;
    const size_t bytes = kStatusBytes + ((wl->counters * sizeof(unsigned) + 255) / 256) * 256 +
                         wl->partial_floats * sizeof(float);
    info->workspace_bytes = (int64_t)bytes;
    return FORGE_OK;
}

// Status word, counters and partials all start from zero.
bool clear_workspace(const Workspace &ws) { return cudaMemset(ws.base, 0, ws.bytes) == cudaSuccess; }

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; prev = -1; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~DeviceGuard()
    {
        int cur = -1;
        if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
    }
};

size_t elem_bytes(const forge_fused_linear_desc_t &d) { return (d.dtype == FORGE_F32 || d.dtype == FORGE_F32_TF32X3) ? 4 : 2; }
size_t out_bytes(const forge_fused_linear_desc_t &d)
{
    if (d.red == FORGE_RED_SUM || d.red == FORGE_RED_MAX || d.red == FORGE_RED_LOGSUMEXP || d.red == FORGE_RED_CROSS_ENTROPY)
        return (size_t)d.M * 4;
    return (size_t)d.M * (size_t)(d.red == FORGE_RED_MEAN_GELU_RESIDUAL ? d.K : d.N) * elem_bytes(d);
}

forge_status_t check_run_args(const Handle &h, const RunArgs &a)
{
    if (!a.X || !a.W || !a.out) return FORGE_ERR_INVALID_ARG;
    if (h.d.has_bias && !a.b) return FORGE_ERR_INVALID_ARG;
    if (h.d.red == FORGE_RED_LAYERNORM && (!a.gamma || !a.beta)) return FORGE_ERR_INVALID_ARG;
    if (h.d.red == FORGE_RED_CROSS_ENTROPY && !a.gamma) return FORGE_ERR_INVALID_ARG;      // the targets
    const uintptr_t m = (uintptr_t)a.X | (uintptr_t)a.W | (uintptr_t)a.out | (uintptr_t)a.b |
                        (uintptr_t)a.gamma | (uintptr_t)a.beta;
    // Operands that travel by TMA and 128-bit accesses need 16-byte alignment.  The FFMA kernel
    // falls back to scalar accesses when unaligned, but still needs element alignment.
    if (h.d.dtype != FORGE_F32 ? (m % 16 != 0) : (m % 4 != 0)) return FORGE_ERR_INVALID_ARG;
    return FORGE_OK;
}

forge_status_t dispatch(Handle &h, const RunArgs &a)
{
    switch (h.info.kernel) {
    case FORGE_KERNEL_F32_FFMA: return k1_launch(h, a);
    case FORGE_KERNEL_BF16_TCGEN05: return k2_launch(h, a);
    case FORGE_KERNEL_BF16_SKINNY: return k3_launch(h, a);
    case FORGE_KERNEL_BF16_TCGEN05_LN: return k4_launch(h, a);
    case FORGE_KERNEL_F32_TF32X3: return k5_launch(h, a);
    }
    return FORGE_ERR_UNSUPPORTED;
}

}  // namespace

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static forge_status_t encode_tmap(CUtensorMap *tm, CUtensorMapDataType type, size_t elem, const void *ptr, uint64_t rows,
                                  uint64_t cols, uint32_t box_rows, uint32_t box_cols)
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *sym = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &sym, 12000, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess || !sym)
            return FORGE_ERR_CUDA;
        fn = (EncodeTiledFn)sym;
    }
    const cuuint64_t dims[2] = {cols, rows};                  // innermost first
    const cuuint64_t strides[1] = {cols * elem};              // bytes, dimension 1
    const cuuint32_t box[2] = {box_cols, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    // L2 fetch granularity of the tensor maps: 256 bytes measured best; a tuning build may set
    // -DFORGE_TMA_L2_PROMOTION=0|64|128|256
#ifndef FORGE_TMA_L2_PROMOTION
#define FORGE_TMA_L2_PROMOTION 256
#endif
    constexpr int promo = FORGE_TMA_L2_PROMOTION;
    const CUtensorMapL2promotion l2 = promo == 0 ? CU_TENSOR_MAP_L2_PROMOTION_NONE
                                      : promo == 64 ? CU_TENSOR_MAP_L2_PROMOTION_L2_64B
                                      : promo == 128 ? CU_TENSOR_MAP_L2_PROMOTION_L2_128B
                                                     : CU_TENSOR_MAP_L2_PROMOTION_L2_256B;
    const CUresult r = fn(tm, type, 2, const_cast<void *>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                          CU_TENSOR_MAP_SWIZZLE_128B, l2, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? FORGE_OK : FORGE_ERR_CUDA;
}

forge_status_t encode_tmap_16(CUtensorMap *tm, const void *ptr, uint64_t rows, uint64_t cols,
                              uint32_t box_rows, uint32_t box_cols, int f16)
{
    return encode_tmap(tm, f16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, ptr, rows, cols, box_rows, box_cols);
}

forge_status_t encode_tmap_f32(CUtensorMap *tm, const void *ptr, uint64_t rows, uint64_t cols,
                               uint32_t box_rows, uint32_t box_cols)
{
    return encode_tmap(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, ptr, rows, cols, box_rows, box_cols);
}

}  // namespace forge

using namespace forge;

// One CTA, one barrier that nothing ever signals: the bounded wait must give up after
// `budget_ns`, leave (FORGE_ERR_TIMEOUT, site, detail, CTA, thread) in the status area and
// let the kernel end normally.
__global__ void forge_wait_selftest_kernel(int *status, unsigned long long budget_ns, int detail)
{
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        ptx::mbar_init(&bar, 1);
        ptx::fence_mbar_init();
    }
    __syncthreads();
    if (threadIdx.x == 32) ptx::mbar_wait(&bar, 0, status, SITE_TMA_FULL, detail, budget_ns);
}

// Register-only fused multiply-add loop: 16 independent packed-pair chains per thread, nothing but
// FMA-pipe work in the loop body.  What it sustains is the ceiling of any FFMA kernel on this device
// at the clock the device actually holds under that load.
__global__ void __launch_bounds__(512, 2) forge_ffma_rate_kernel(float *sink, float a0, float b0, int iters)
{
    unsigned long long acc[16], a, b;
    asm("mov.b64 %0, {%1, %1};" : "=l"(a) : "f"(a0));
    asm("mov.b64 %0, {%1, %1};" : "=l"(b) : "f"(b0));
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const float v = (float)(threadIdx.x + i);
        asm("mov.b64 %0, {%1, %1};" : "=l"(acc[i]) : "f"(v));
    }
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int u = 0; u < 4; ++u)
#pragma unroll
            for (int i = 0; i < 16; ++i) asm volatile("fma.rn.f32x2 %0, %0, %1, %2;" : "+l"(acc[i]) : "l"(a), "l"(b));
    }
    unsigned long long x = 0;
#pragma unroll
    for (int i = 0; i < 16; ++i) x ^= acc[i];
    if (x == 0x7ff0dead7ff0beefull) sink[0] = 1.f;      // keeps the chains alive; practically never true
}

// Load-only stream: one thread per CTA keeps `stages` contiguous bulk copies of `piece` bytes in flight into a ring
// of shared memory (global -> shared, completion counted in bytes on an mbarrier per slot); nothing is computed.
// What it sustains is what the memory system delivers to a kernel that only reads.
__global__ void __launch_bounds__(32, 1) forge_read_stream_kernel(const uint8_t *src, size_t bytes, uint32_t piece, int stages, int *status)
{
    extern __shared__ uint8_t stream_raw[];
    uint8_t *ring = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(stream_raw) + 127) & ~uintptr_t(127));
    __shared__ uint64_t full[8];
    if (threadIdx.x == 0) {
        for (int i = 0; i < stages; ++i) ptx::mbar_init(&full[i], 1);
        ptx::fence_mbar_init();
    }
    __syncthreads();
    if (threadIdx.x != 0) return;
    const size_t pieces = bytes / piece;
    const size_t lo = pieces * blockIdx.x / gridDim.x, hi = pieces * (blockIdx.x + 1) / gridDim.x;
    long long issued = 0;
    bool ok = true;
    for (size_t i = lo; i < hi && ok; ++i, ++issued) {
        const int slot = (int)(issued % stages);
        // the slot's previous copy must have landed before it is overwritten
        if (issued >= stages && !ptx::mbar_wait(&full[slot], (uint32_t)((issued / stages - 1) & 1), status, SITE_TMA_FULL, slot)) { ok = false; break; }
        ptx::mbar_expect_tx(&full[slot], piece);
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(ptx::smem_u32(ring + (size_t)slot * piece)), "l"(src + i * piece), "r"(piece), "r"(ptx::smem_u32(&full[slot])) : "memory");
    }
    // every copy still in flight lands before the CTA leaves
    for (long long j = issued > stages ? issued - stages : 0; j < issued && ok; ++j)
        ok = ptx::mbar_wait(&full[(int)(j % stages)], (uint32_t)((j / stages) & 1), status, SITE_TMA_FULL, (int)(j % stages));
    if (!ok) __nanosleep(500000);
}

extern "C" {

forge_status_t forge_selftest_read_stream(int device, double *gbs_back_to_back, double *gbs_single)
{
    if (!gbs_back_to_back || device < 0) return FORGE_ERR_INVALID_ARG;
    DeviceGuard g(device);
    if (!g.ok) return FORGE_ERR_CUDA;
    int sms = 0, major = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || sms <= 0 ||
        cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess || major != 10)
        return FORGE_ERR_CUDA;
    constexpr size_t kPart = (size_t)256 << 20;          // one "weight": twice the L2
    constexpr int kParts = 3, kStages = 4;
    constexpr uint32_t kPiece = 32768;
    constexpr size_t kSmem = (size_t)kStages * kPiece + 128;
    uint8_t *buf = nullptr;
    int *status = nullptr;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    if (cudaMalloc(&buf, kParts * kPart) != cudaSuccess || cudaMalloc(&status, 256) != cudaSuccess) {
        cudaGetLastError();
        cudaFree(buf);
        return FORGE_ERR_ALLOC;
    }
    forge_status_t st = FORGE_ERR_CUDA;
    bool ok = cudaMemset(buf, 1, kParts * kPart) == cudaSuccess && cudaMemset(status, 0, 256) == cudaSuccess &&
              cudaFuncSetAttribute(forge_read_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmem) == cudaSuccess &&
              cudaEventCreate(&e0) == cudaSuccess && cudaEventCreate(&e1) == cudaSuccess;
    auto launch = [&](int i) { forge_read_stream_kernel<<<sms, 32, kSmem>>>(buf + (size_t)(i % kParts) * kPart, kPart, kPiece, kStages, status); };
    float ms = 0.f;
    if (ok) {
        constexpr int kRuns = 30;
        for (int i = 0; i < kParts; ++i) launch(i);
        ok = cudaDeviceSynchronize() == cudaSuccess && cudaEventRecord(e0) == cudaSuccess;
        for (int i = 0; i < kRuns; ++i) launch(i);
        ok = ok && cudaEventRecord(e1) == cudaSuccess && cudaEventSynchronize(e1) == cudaSuccess &&
             cudaEventElapsedTime(&ms, e0, e1) == cudaSuccess && ms > 0.f;
        if (ok) *gbs_back_to_back = (double)kPart * kRuns / (ms * 1e-3) / 1e9;
    }
    if (ok && gbs_single) {
        float best[11];
        for (int i = 0; i < 11 && ok; ++i) {
            ok = cudaEventRecord(e0) == cudaSuccess;
            launch(i);
            ok = ok && cudaEventRecord(e1) == cudaSuccess && cudaEventSynchronize(e1) == cudaSuccess &&
                 cudaEventElapsedTime(&best[i], e0, e1) == cudaSuccess;
        }
        if (ok) {
            for (int i = 0; i < 11; ++i)
                for (int j = i + 1; j < 11; ++j)
                    if (best[j] < best[i]) { const float t = best[i]; best[i] = best[j]; best[j] = t; }
            *gbs_single = (double)kPart / (best[5] * 1e-3) / 1e9;          // the median launch
        }
    }
    int word = 0;
    if (ok && cudaMemcpy(&word, status, sizeof(word), cudaMemcpyDeviceToHost) == cudaSuccess) st = word == 0 ? FORGE_OK : (forge_status_t)(word >> 16);
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    cudaFree(buf);
    cudaFree(status);
    if (!ok) cudaGetLastError();
    return st;
}

forge_status_t forge_selftest_ffma_rate(int device, int milliseconds, double *tflops, double *sm_mhz_effective)
{
    if (!tflops || milliseconds <= 0 || milliseconds > 2000 || device < 0) return FORGE_ERR_INVALID_ARG;
    DeviceGuard g(device);
    if (!g.ok) return FORGE_ERR_CUDA;
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || sms <= 0) return FORGE_ERR_CUDA;
    float *sink = nullptr;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    if (cudaMalloc(&sink, 256) != cudaSuccess) { cudaGetLastError(); return FORGE_ERR_ALLOC; }
    forge_status_t st = FORGE_ERR_CUDA;
    if (cudaEventCreate(&e0) == cudaSuccess && cudaEventCreate(&e1) == cudaSuccess) {
        const int grid = 2 * sms, threads = 512;
        // calibrate on a short launch, then size one launch for the requested duration
        int iters = 2048;
        float ms = 0.f;
        bool ok = true;
        for (int pass = 0; pass < 2 && ok; ++pass) {
            ok = cudaEventRecord(e0) == cudaSuccess;
            forge_ffma_rate_kernel<<<grid, threads>>>(sink, 0.999f, 1e-3f, iters);
            ok = ok && cudaGetLastError() == cudaSuccess && cudaEventRecord(e1) == cudaSuccess &&
                 cudaEventSynchronize(e1) == cudaSuccess && cudaEventElapsedTime(&ms, e0, e1) == cudaSuccess && ms > 0.f;
            if (ok && pass == 0) {
                const double want = (double)iters * milliseconds / ms;
                iters = want > 1e8 ? 100000000 : (want < 1024 ? 1024 : (int)want);
            }
        }
        if (ok) {
            const double fmas = (double)grid * threads * (double)iters * 4 * 16 * 2;      // two lanes per packed instruction
            *tflops = 2.0 * fmas / (ms * 1e-3) / 1e12;
            if (sm_mhz_effective) *sm_mhz_effective = fmas / (ms * 1e-3) / ((double)sms * 128.0) / 1e6;
            st = FORGE_OK;
        }
    }
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    cudaFree(sink);
    return st;
}

forge_status_t forge_selftest_bounded_wait(int device, int budget_ms, int detail[4])
{
    if (!detail || budget_ms <= 0 || budget_ms > 1000 || device < 0) return FORGE_ERR_INVALID_ARG;
    DeviceGuard g(device);
    if (!g.ok) return FORGE_ERR_CUDA;
    int *status = nullptr;
    if (cudaMalloc(&status, 256) != cudaSuccess) { cudaGetLastError(); return FORGE_ERR_ALLOC; }
    forge_status_t st = FORGE_ERR_CUDA;
    int word[4] = {0, 0, 0, 0};
    if (cudaMemset(status, 0, 256) == cudaSuccess) {
        forge_wait_selftest_kernel<<<1, 64>>>(status, (unsigned long long)budget_ms * 1000000ull, 0x5a5a);
        if (cudaGetLastError() == cudaSuccess && cudaDeviceSynchronize() == cudaSuccess &&
            cudaMemcpy(word, status, sizeof(word), cudaMemcpyDeviceToHost) == cudaSuccess) {
            st = (forge_status_t)(word[0] >> 16);
            detail[0] = word[0] & 0xffff;
            detail[1] = word[1];
            detail[2] = word[2];
            detail[3] = word[3];
        }
    }
    cudaFree(status);
    return st;
}

forge_status_t forge_fused_linear_query_plan(const forge_fused_linear_desc_t *desc, int sm_count, forge_plan_info_t *info)
{
    if (!desc || !info) return FORGE_ERR_INVALID_ARG;
    WorkspaceLayout wl;
    return plan_for(*desc, sm_count, info, &wl);
}

forge_status_t forge_fused_linear_create(const forge_fused_linear_desc_t *desc, forge_fused_linear_t *out)
{
    if (out) *out = nullptr;
    if (!desc || !out) return FORGE_ERR_INVALID_ARG;
    // argument errors are reported before the device is touched
    forge_plan_info_t probe;
    WorkspaceLayout wl;
    forge_status_t st = plan_for(*desc, 148, &probe, &wl);
    if (st != FORGE_OK) return st;

    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || desc->device >= ndev) { cudaGetLastError(); return FORGE_ERR_CUDA; }
    int major = 0, sms = 0, l2 = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, desc->device) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, desc->device) != cudaSuccess ||
        cudaDeviceGetAttribute(&l2, cudaDevAttrL2CacheSize, desc->device) != cudaSuccess)
        return FORGE_ERR_CUDA;
    if (major != 10) return FORGE_ERR_CUDA;     // the kernels are sm_100a only

    Handle *h = new (std::nothrow) Handle();
    if (!h) return FORGE_ERR_ALLOC;
    h->d = *desc;
    h->sm_count = sms;
    h->l2_bytes = l2;
    st = plan_for(*desc, sms, &h->info, &wl);
    if (st != FORGE_OK) { delete h; return st; }

    DeviceGuard g(desc->device);
    if (!g.ok) { delete h; return FORGE_ERR_CUDA; }
    h->ws.bytes = (size_t)h->info.workspace_bytes;
    if (cudaMalloc(&h->ws.base, h->ws.bytes) != cudaSuccess) { cudaGetLastError(); delete h; return FORGE_ERR_ALLOC; }
    char *base = (char *)h->ws.base;
    h->ws.status = (int *)base;
    h->ws.counters = (unsigned *)(base + kStatusBytes);
    h->ws.partial = (float *)(base + kStatusBytes + ((wl.counters * sizeof(unsigned) + 255) / 256) * 256);
    h->ws.partial_floats = (long long)wl.partial_floats;
    h->ws.counter_words = (long long)wl.counters;
    if (!clear_workspace(h->ws)) { cudaFree(h->ws.base); delete h; return FORGE_ERR_CUDA; }

    switch (h->info.kernel) {
    case FORGE_KERNEL_F32_FFMA: st = k1_setup(*h); break;
    case FORGE_KERNEL_BF16_TCGEN05: st = k2_setup(*h); break;
    case FORGE_KERNEL_BF16_SKINNY: st = k3_setup(*h); break;
    case FORGE_KERNEL_BF16_TCGEN05_LN: st = k4_setup(*h); break;
    case FORGE_KERNEL_F32_TF32X3: st = k5_setup(*h); break;
    }
    if (st != FORGE_OK) { cudaFree(h->ws.base); delete h; return st; }
    *out = reinterpret_cast<forge_fused_linear_t>(h);
    return FORGE_OK;
}

forge_status_t forge_fused_linear_run(forge_fused_linear_t hh, const void *X, const void *W, const void *b,
                                      const void *gamma, const void *beta, void *out, void *cuda_stream)
{
    if (!hh) return FORGE_ERR_INVALID_ARG;
    Handle &h = *reinterpret_cast<Handle *>(hh);
    RunArgs a{X, W, h.d.has_bias ? b : nullptr, gamma, beta, out, (cudaStream_t)cuda_stream};
    const forge_status_t st = check_run_args(h, a);
    if (st != FORGE_OK) return st;
    DeviceGuard g(h.d.device);
    if (!g.ok) return FORGE_ERR_CUDA;
    return dispatch(h, a);
}

// Block plan of the pipelined host path: 256-row multiples (whole CTA-pair tiles), at most
// kHostPipeMaxBlocks blocks, and only when X is large enough for the overlap to matter.
static int64_t host_block_rows(const forge_fused_linear_desc_t &d)
{
    const size_t bx = (size_t)d.M * (size_t)d.K * elem_bytes(d);
    if (d.M < 1024 || bx < ((size_t)8 << 20)) return 0;
    const int64_t want = (d.M + kHostPipeMaxBlocks - 1) / kHostPipeMaxBlocks;
    return ((want + 255) / 256) * 256;
}

static void pipeline_free(HostPipeline *p)
{
    if (!p) return;
    if (p->block) forge_fused_linear_destroy(reinterpret_cast<forge_fused_linear_t>(p->block));
    if (p->last) forge_fused_linear_destroy(reinterpret_cast<forge_fused_linear_t>(p->last));
    for (int i = 0; i < kHostPipeMaxBlocks; ++i) {
        if (p->landed[i]) cudaEventDestroy(p->landed[i]);
        if (p->computed[i]) cudaEventDestroy(p->computed[i]);
    }
    if (p->s_in) cudaStreamDestroy(p->s_in);
    if (p->s_run) cudaStreamDestroy(p->s_run);
    if (p->s_out) cudaStreamDestroy(p->s_out);
    delete p;
}

static forge_status_t pipeline_create(Handle &h, int64_t block_rows)
{
    HostPipeline *p = new (std::nothrow) HostPipeline();
    if (!p) return FORGE_ERR_ALLOC;
    p->block_rows = block_rows;
    p->blocks = (int)((h.d.M + block_rows - 1) / block_rows);
    forge_status_t st = FORGE_OK;
    if (cudaStreamCreateWithFlags(&p->s_in, cudaStreamNonBlocking) != cudaSuccess ||
        cudaStreamCreateWithFlags(&p->s_run, cudaStreamNonBlocking) != cudaSuccess ||
        cudaStreamCreateWithFlags(&p->s_out, cudaStreamNonBlocking) != cudaSuccess)
        st = FORGE_ERR_CUDA;
    for (int i = 0; i < p->blocks && st == FORGE_OK; ++i)
        if (cudaEventCreateWithFlags(&p->landed[i], cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&p->computed[i], cudaEventDisableTiming) != cudaSuccess)
            st = FORGE_ERR_CUDA;
    forge_fused_linear_desc_t d = h.d;
    if (st == FORGE_OK) {
        d.M = block_rows;
        st = forge_fused_linear_create(&d, reinterpret_cast<forge_fused_linear_t *>(&p->block));
    }
    const int64_t rest = h.d.M - (int64_t)(p->blocks - 1) * block_rows;
    if (st == FORGE_OK && rest != block_rows) {
        d.M = rest;
        st = forge_fused_linear_create(&d, reinterpret_cast<forge_fused_linear_t *>(&p->last));
    }
    if (st != FORGE_OK) { cudaGetLastError(); pipeline_free(p); return st; }
    h.pipe = p;
    return FORGE_OK;
}

forge_status_t forge_fused_linear_run_host(forge_fused_linear_t hh, const void *X, const void *W, const void *b,
                                           const void *gamma, const void *beta, void *out)
{
    if (!hh) return FORGE_ERR_INVALID_ARG;
    Handle &h = *reinterpret_cast<Handle *>(hh);
    const forge_fused_linear_desc_t &d = h.d;
    if (!X || !W || !out || (d.has_bias && !b) || (d.red == FORGE_RED_LAYERNORM && (!gamma || !beta)) ||
        (d.red == FORGE_RED_CROSS_ENTROPY && !gamma))
        return FORGE_ERR_INVALID_ARG;
    DeviceGuard g(d.device);
    if (!g.ok) return FORGE_ERR_CUDA;
    const size_t e = elem_bytes(d);
    const size_t bx = (size_t)d.M * d.K * e, bw = (size_t)d.N * d.K * e, bn = (size_t)d.N * e, bo = out_bytes(d);
    const size_t bt = (size_t)d.M * 4;                       // int32 targets of the cross-entropy
    const size_t bg = bn > bt ? bn : bt;                     // the gamma slot holds either
    if (!h.hX) {
        if (cudaMalloc(&h.hX, bx) != cudaSuccess || cudaMalloc(&h.hW, bw) != cudaSuccess ||
            cudaMalloc(&h.hb, bn) != cudaSuccess || cudaMalloc(&h.hg, bg) != cudaSuccess ||
            cudaMalloc(&h.hbe, bn) != cudaSuccess || cudaMalloc(&h.hout, bo) != cudaSuccess) {
            cudaGetLastError();
            cudaFree(h.hX); cudaFree(h.hW); cudaFree(h.hb); cudaFree(h.hg); cudaFree(h.hbe); cudaFree(h.hout);
            h.hX = h.hW = h.hb = h.hg = h.hbe = h.hout = nullptr;
            return FORGE_ERR_ALLOC;
        }
        const int64_t block_rows = host_block_rows(d);
        if (block_rows > 0 && block_rows < d.M) {
            const forge_status_t st = pipeline_create(h, block_rows);
            if (st != FORGE_OK) return st;
        }
    }
    HostPipeline *pp = h.pipe;
    cudaStream_t s = pp ? pp->s_in : nullptr;
    const bool has_sub = d.red == FORGE_RED_MEAN_GELU_RESIDUAL && gamma;
    const bool has_tgt = d.red == FORGE_RED_CROSS_ENTROPY;
    // everything but X first: the first block of rows needs all of W
    bool ok = cudaMemcpyAsync(h.hW, W, bw, cudaMemcpyHostToDevice, s) == cudaSuccess;
    if (ok && d.has_bias) ok = cudaMemcpyAsync(h.hb, b, bn, cudaMemcpyHostToDevice, s) == cudaSuccess;
    if (ok && d.red == FORGE_RED_LAYERNORM)
        ok = cudaMemcpyAsync(h.hg, gamma, bn, cudaMemcpyHostToDevice, s) == cudaSuccess &&
             cudaMemcpyAsync(h.hbe, beta, bn, cudaMemcpyHostToDevice, s) == cudaSuccess;
    if (ok && has_sub) ok = cudaMemcpyAsync(h.hg, gamma, bn, cudaMemcpyHostToDevice, s) == cudaSuccess;
    if (ok && has_tgt) ok = cudaMemcpyAsync(h.hg, gamma, bt, cudaMemcpyHostToDevice, s) == cudaSuccess;
    // after the first enqueue no path returns before the stream has drained: a copy still in flight
    // would go on reading the caller's buffers (or writing `out`) after the call has returned
    if (!ok) { cudaStreamSynchronize(s); return FORGE_ERR_CUDA; }
    const void *aux = (d.red == FORGE_RED_LAYERNORM || has_sub || has_tgt) ? h.hg : nullptr;

    if (!pp) {
        forge_status_t st = cudaMemcpyAsync(h.hX, X, bx, cudaMemcpyHostToDevice, s) == cudaSuccess ? FORGE_OK : FORGE_ERR_CUDA;
        if (st == FORGE_OK) {
            RunArgs a{h.hX, h.hW, d.has_bias ? h.hb : nullptr, aux, h.hbe, h.hout, s};
            st = dispatch(h, a);
        }
        if (st == FORGE_OK && cudaMemcpyAsync(out, h.hout, bo, cudaMemcpyDeviceToHost, s) != cudaSuccess) st = FORGE_ERR_CUDA;
        const bool drained = cudaStreamSynchronize(s) == cudaSuccess;
        return st != FORGE_OK ? st : (drained ? FORGE_OK : FORGE_ERR_CUDA);
    }

    // Blocks of rows: every reduction here runs along N, so a block of rows is a complete problem.
    const size_t x_row = (size_t)d.K * e, o_row = bo / (size_t)d.M;
    forge_status_t st = FORGE_OK;
    for (int i = 0; i < pp->blocks && st == FORGE_OK; ++i) {
        const int64_t r0 = (int64_t)i * pp->block_rows;
        const int64_t rows = (i == pp->blocks - 1) ? d.M - r0 : pp->block_rows;
        Handle &hb = (i == pp->blocks - 1 && pp->last) ? *pp->last : *pp->block;
        char *xd = (char *)h.hX + (size_t)r0 * x_row, *od = (char *)h.hout + (size_t)r0 * o_row;
        ok = cudaMemcpyAsync(xd, (const char *)X + (size_t)r0 * x_row, (size_t)rows * x_row, cudaMemcpyHostToDevice, pp->s_in) == cudaSuccess &&
             cudaEventRecord(pp->landed[i], pp->s_in) == cudaSuccess &&
             cudaStreamWaitEvent(pp->s_run, pp->landed[i], 0) == cudaSuccess;
        if (!ok) { st = FORGE_ERR_CUDA; break; }
        // per-row auxiliary data (the cross-entropy targets) moves with the block; per-column data does not
        const void *aux_i = has_tgt ? (const void *)((const char *)h.hg + (size_t)r0 * 4) : aux;
        RunArgs a{xd, h.hW, d.has_bias ? h.hb : nullptr, aux_i, h.hbe, od, pp->s_run};
        st = dispatch(hb, a);
        if (st != FORGE_OK) break;
        ok = cudaEventRecord(pp->computed[i], pp->s_run) == cudaSuccess &&
             cudaStreamWaitEvent(pp->s_out, pp->computed[i], 0) == cudaSuccess &&
             cudaMemcpyAsync((char *)out + (size_t)r0 * o_row, od, (size_t)rows * o_row, cudaMemcpyDeviceToHost, pp->s_out) == cudaSuccess;
        if (!ok) st = FORGE_ERR_CUDA;
    }
    // drain all three streams whatever happened, so that no copy still reads the caller's buffers
    const bool drained = cudaStreamSynchronize(pp->s_in) == cudaSuccess && cudaStreamSynchronize(pp->s_run) == cudaSuccess &&
                         cudaStreamSynchronize(pp->s_out) == cudaSuccess;
    if (st != FORGE_OK) return st;
    if (!drained) return FORGE_ERR_CUDA;
    // a give-up inside a block's kernel is recorded in the child's status word: fold it into this handle's
    for (Handle *c : {pp->block, pp->last}) {
        if (!c) continue;
        int word = 0;
        if (cudaMemcpy(&word, c->ws.status, sizeof(word), cudaMemcpyDeviceToHost) != cudaSuccess) return FORGE_ERR_CUDA;
        if (word != 0) {
            cudaMemcpy(h.ws.status, c->ws.status, 4 * sizeof(int), cudaMemcpyDeviceToDevice);
            forge_fused_linear_last_status(reinterpret_cast<forge_fused_linear_t>(c));     // clears the child
        }
    }
    return FORGE_OK;
}

forge_status_t forge_fused_linear_last_status(forge_fused_linear_t hh)
{
    if (!hh) return FORGE_ERR_INVALID_ARG;
    Handle &h = *reinterpret_cast<Handle *>(hh);
    DeviceGuard g(h.d.device);
    if (!g.ok) return FORGE_ERR_CUDA;
    if (cudaDeviceSynchronize() != cudaSuccess) return FORGE_ERR_CUDA;
    if (cudaMemcpy(h.last_detail, h.ws.status, sizeof(h.last_detail), cudaMemcpyDeviceToHost) != cudaSuccess) return FORGE_ERR_CUDA;
    const int word = h.last_detail[0];
    if (word != 0) {
        // a give-up may have left arrival counters half way: clear the whole workspace
        clear_workspace(h.ws);
        return (forge_status_t)(word >> 16);
    }
    return FORGE_OK;
}

forge_status_t forge_fused_linear_last_wait_detail(forge_fused_linear_t hh, int detail[4])
{
    if (!hh || !detail) return FORGE_ERR_INVALID_ARG;
    const Handle &h = *reinterpret_cast<Handle *>(hh);
    detail[0] = h.last_detail[0] & 0xffff;
    detail[1] = h.last_detail[1];
    detail[2] = h.last_detail[2];
    detail[3] = h.last_detail[3];
    return FORGE_OK;
}

forge_status_t forge_fused_linear_get_plan(forge_fused_linear_t hh, forge_plan_info_t *info)
{
    if (!hh || !info) return FORGE_ERR_INVALID_ARG;
    *info = reinterpret_cast<Handle *>(hh)->info;
    return FORGE_OK;
}

int forge_fused_linear_launches_per_run(forge_fused_linear_t hh) { return hh ? 1 : 0; }

const char *forge_fused_linear_kernel_name(forge_fused_linear_t hh)
{
    return hh ? forge_kernel_name(reinterpret_cast<Handle *>(hh)->info.kernel) : "no handle";
}

forge_status_t forge_fused_linear_destroy(forge_fused_linear_t hh)
{
    if (!hh) return FORGE_ERR_INVALID_ARG;
    Handle *h = reinterpret_cast<Handle *>(hh);
    {
        DeviceGuard g(h->d.device);
        cudaFree(h->ws.base);
        cudaFree(h->hX); cudaFree(h->hW); cudaFree(h->hb); cudaFree(h->hg); cudaFree(h->hbe); cudaFree(h->hout);
        pipeline_free(h->pipe);
    }
    delete h;
    return FORGE_OK;
}

const char *forge_status_string(forge_status_t s)
{
    switch (s) {
    case FORGE_OK: return "ok";
    case FORGE_ERR_INVALID_ARG: return "invalid argument";
    case FORGE_ERR_UNSUPPORTED: return "unsupported descriptor (no kernel serves it; there is no fallback)";
    case FORGE_ERR_CUDA: return "CUDA error or no sm_100 device";
    case FORGE_ERR_ALLOC: return "allocation failed";
    case FORGE_ERR_TIMEOUT: return "a bounded device-side wait expired";
    case FORGE_ERR_SCRATCH_LIMIT: return "problem needs more scratch than the fixed no-allocation buffer holds";
    case FORGE_ERR_BOUNDS: return "bounds-checked build: an index outside its allocation (the access was skipped)";
    }
    return "unknown status";
}

const char *forge_kernel_name(forge_kernel_t k)
{
    switch (k) {
    case FORGE_KERNEL_F32_FFMA: return "f32_ffma_128x128x16";
    case FORGE_KERNEL_BF16_TCGEN05: return "bf16_tcgen05_tma";
    case FORGE_KERNEL_BF16_SKINNY: return "bf16_skinny_swapab_tcgen05";
    case FORGE_KERNEL_BF16_TCGEN05_LN: return "bf16_tcgen05_tma_layernorm";
    case FORGE_KERNEL_F32_TF32X3: return "f32_tf32x3_tcgen05_tma";
    }
    return "unknown kernel";
}

}  // extern "C"
