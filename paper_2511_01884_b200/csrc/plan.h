// Host-side plan shared by the C interface and the per-kernel launchers.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/forge.h"

namespace forge {

struct RunArgs {
    const void *X, *W, *b, *gamma, *beta;
    void *out;
    cudaStream_t stream;
};

// Device scratch owned by a handle.
struct Workspace {
    float *partial = nullptr;        // per-tile row partials (sum/max), fp32
    unsigned *counters = nullptr;    // arrival counters, zero between runs
    int *status = nullptr;           // status word
    void *base = nullptr;            // the single allocation the three point into
    size_t bytes = 0;
    long long partial_floats = 0, counter_words = 0;     // extents of the two areas (for the bounds-checked build)
};

struct Handle;
constexpr int kHostPipeMaxBlocks = 8;
struct HostPipeline {
    cudaStream_t s_in = nullptr, s_run = nullptr, s_out = nullptr;
    cudaEvent_t landed[kHostPipeMaxBlocks] = {}, computed[kHostPipeMaxBlocks] = {};
    Handle *block = nullptr, *last = nullptr;      // child handles (last: nullptr if all blocks are equal)
    int64_t block_rows = 0;
    int blocks = 0;
};

struct Handle {
    forge_fused_linear_desc_t d;
    forge_plan_info_t info;
    int sm_count = 0;
    int l2_bytes = 0;
    int last_detail[4] = {0, 0, 0, 0};   // status area as read by the last last_status() call
    Workspace ws;
    // staging buffers of run_host()
    void *hX = nullptr, *hW = nullptr, *hb = nullptr, *hg = nullptr, *hbe = nullptr, *hout = nullptr;
    // run_host() on a large problem walks X in blocks of rows so that the upload of block i+1, the
    // kernel on block i and the download of block i-1 overlap: three streams, one event pair per
    // block, and a child handle planned for a block's rows (plus one for a shorter last block).
    HostPipeline *pipe = nullptr;
    // cached TMA descriptors (bf16 kernels): re-encoded only when a pointer changes
    CUtensorMap tmX, tmW, tmY;
    const void *tmX_ptr = nullptr, *tmW_ptr = nullptr, *tmY_ptr = nullptr;
};

// K serpentine (tensor-core kernels): every other tile of a unit walks K downwards.  All units turn round at about the
// same time, and a wave reads the X panels of the same group of rows as the wave before it, so what was read last is
// read first, while it is still in L2.  It pays only when the operands of one wave (the group's rows of X and the
// columns of W that the units cover meanwhile, over all K) do not fit in L2 anyway -- in half of it, since the two
// dies each cache what both read: C3 (72 MB a wave) reads 15 % less from DRAM and runs 1.9 % faster; with K = 4096
// (36 MB) the turn costs 0.5-1 %.  group_rows = 0: the tiles of a row strip are neighbours in the schedule (LayerNorm).
inline bool k_serpentine_pays(const forge_fused_linear_desc_t &d, int64_t units, int unit_rows, int unit_cols,
                              int64_t group_rows, int elem_bytes, int l2_bytes)
{
    if (units <= 0) return false;
    const int64_t tiles_n = (d.N + unit_cols - 1) / unit_cols;
    int64_t rows_x = group_rows > 0 ? group_rows : (units + tiles_n - 1) / tiles_n * unit_rows;
    if (rows_x > d.M) rows_x = d.M;
    const int64_t units_per_column = (rows_x + unit_rows - 1) / unit_rows;
    int64_t cols_w = (units + units_per_column - 1) / units_per_column * unit_cols;
    if (cols_w > d.N) cols_w = d.N;
    return (rows_x + cols_w) * d.K * elem_bytes > (int64_t)l2_bytes / 2;
}

// Kernels whose CTAs wait on one another are launched cooperatively (all CTAs resident at once).
// A profiling build (-DFORGE_PROFILING_NO_COOPERATIVE) drops the attribute, because profilers
// refuse cooperative launches of clusters; it is not for production use: the grids never exceed
// the SM count and every wait is bounded, so the worst case on a GPU that is busy with other work
// is a reported time-out, not a hang, but co-residency is no longer guaranteed.
constexpr bool cooperative_launch_enabled()
{
#ifdef FORGE_PROFILING_NO_COOPERATIVE
    return false;
#else
    return true;
#endif
}

// Layout of the workspace (element counts) for a plan; filled by the planners.
struct WorkspaceLayout {
    size_t partial_floats = 0;
    size_t counters = 0;
};

// Each kernel family: a host-only planner (no device access), a one-time setup on the
// device (function attributes), and a launcher.
forge_status_t k1_plan(const forge_fused_linear_desc_t &d, int sm_count, forge_plan_info_t *info, WorkspaceLayout *wl);
forge_status_t k1_setup(Handle &h);
forge_status_t k1_launch(Handle &h, const RunArgs &a);

forge_status_t k2_plan(const forge_fused_linear_desc_t &d, int sm_count, forge_plan_info_t *info, WorkspaceLayout *wl);
forge_status_t k2_setup(Handle &h);
forge_status_t k2_launch(Handle &h, const RunArgs &a);

forge_status_t k3_plan(const forge_fused_linear_desc_t &d, int sm_count, forge_plan_info_t *info, WorkspaceLayout *wl);
forge_status_t k3_setup(Handle &h);
forge_status_t k3_launch(Handle &h, const RunArgs &a);

forge_status_t k4_plan(const forge_fused_linear_desc_t &d, int sm_count, forge_plan_info_t *info, WorkspaceLayout *wl);
forge_status_t k4_setup(Handle &h);
forge_status_t k4_launch(Handle &h, const RunArgs &a);

forge_status_t k5_plan(const forge_fused_linear_desc_t &d, int sm_count, forge_plan_info_t *info, WorkspaceLayout *wl);
forge_status_t k5_setup(Handle &h);
forge_status_t k5_launch(Handle &h, const RunArgs &a);

// Encode a 2-D row-major tensor map [rows, cols] of 16-bit elements (bfloat16, or IEEE half if
// f16 != 0) with a [box_rows, box_cols] box and the 128-byte shared-memory swizzle.  Host-only
// driver call.
forge_status_t encode_tmap_16(CUtensorMap *tm, const void *ptr, uint64_t rows, uint64_t cols,
                              uint32_t box_rows, uint32_t box_cols, int f16);

// The same for fp32 elements (box_cols = 32 gives the 128-byte rows of the swizzle).
forge_status_t encode_tmap_f32(CUtensorMap *tm, const void *ptr, uint64_t rows, uint64_t cols,
                               uint32_t box_rows, uint32_t box_cols);

}  // namespace forge
