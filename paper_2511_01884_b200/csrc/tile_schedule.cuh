// The schedule of the persistent tensor-core kernels (16-bit and TF32x3): which output tile a unit (a CTA, or a
// pair of CTAs) works on next, the cut of the last wave along K, and -- on the host -- the grid and the layout of
// the handle's workspace that go with it.  One copy for both kernels; they differ in tile sizes only.
#pragma once

#include <stdint.h>
#include <stddef.h>

#include "common.cuh"

namespace forge {

// One item of a unit's work list: a tile and a range of k-blocks.  Unit c of C takes the whole tiles c, c + C, ...
// of the full waves and then at most one item of the last wave.  When the tiles left for the last wave are at most
// half the units, each is cut along K into S parts that run on S units at once: parts 1..S-1 leave their raw
// accumulators in a scratch area and count themselves in; part 0 waits for them (bounded), adds them into its
// accumulator in part order and runs the epilogue.  The same cut lets a problem with fewer tiles than SMs stream its
// weights with most of the GPU.
struct TileItem {
    int tm, tn;                 // row unit (a tile's or a pair tile's rows), 256-column tile
    int kb_lo, kb_hi;           // k-blocks [kb_lo, kb_hi)
    int part, tail;             // part of the K split (0 leads), index of the tile among the split ones (-1: whole tile)
    int pass;                   // LayerNorm of rows wider than the grid: 0 = statistics only, 1 = normalise and store
};

// Tile index -> (row unit, column tile).  group_m <= 0: the N-tiles of a row strip are neighbours in the schedule
// (LayerNorm: they wait for one another).  Otherwise tiles are walked in groups of group_m row units, so that a wave's
// operands stay in L2; with REVERSE_ODD every other group walks the N-tiles backwards: the W panels last used are
// still in L2 when the next group starts.
template <bool REVERSE_ODD>
__device__ __forceinline__ void tile_coords(int t, int units_m, int tiles_n, int group_m, int &tm, int &tn)
{
    if (group_m <= 0) {
        tm = t / tiles_n;
        tn = t - tm * tiles_n;
        return;
    }
    const int group_size = group_m * tiles_n;
    const int g = t / group_size, r = t - g * group_size;
    const int gm = min(group_m, units_m - g * group_m);
    tm = g * group_m + r % gm;
    tn = r / gm;
    if (REVERSE_ODD && (g & 1)) tn = tiles_n - 1 - tn;
}

// Item j of unit `unit` of `units`; false when the list is exhausted.  two_pass: every tile twice, the unit's whole
// list once for the statistics, then once more to normalise.
template <bool REVERSE_ODD>
__device__ __forceinline__ bool schedule_item(int j, int unit, int units, int units_m, int tiles_n, int num_kb, int tail_parts,
                                              int tail_kb, bool two_pass, int group_m, TileItem &w)
{
    const int total = units_m * tiles_n, full = total / units, rest = total - full * units;
    int t;
    w.kb_lo = 0;
    w.kb_hi = num_kb;
    w.part = 0;
    w.tail = -1;
    w.pass = 0;
    if (two_pass) {
        const int mine = full + (unit < rest ? 1 : 0);
        if (j >= mine) { j -= mine; w.pass = 1; }
    }
    if (j < full) {
        t = j * units + unit;
    } else if (j == full && tail_parts <= 1) {
        if (unit >= rest) return false;
        t = full * units + unit;
    } else if (j == full) {
        if (unit >= rest * tail_parts) return false;
        w.tail = unit / tail_parts;
        w.part = unit - w.tail * tail_parts;
        t = full * units + w.tail;
        w.kb_lo = w.part * tail_kb;
        w.kb_hi = min(w.kb_lo + tail_kb, num_kb);
    } else {
        return false;
    }
    tile_coords<REVERSE_ODD>(t, units_m, tiles_n, group_m, w.tm, w.tn);
    return true;
}

// ---- host side: grid, K split of the last wave and workspace layout -- a pure function of the problem and the SM
// count, used by the planners and by the launchers ----
constexpr int kTailMaxParts = 8;         // bounds the scratch area and the serial adds of part 0
constexpr int kTailMaxFullWaves = 8;     // after that many full waves the last one is too small a share to matter
                                         // (55 waves: measured 3 % slower with the cut than without)
constexpr int kEpiGroupThreads = 128;    // threads of an epilogue group: one per row of a half tile

struct ScheduleLayout {
    int64_t tiles_m, tiles_n, units, slots, ctas;      // slots: units the GPU offers; ctas: units launched
    int tail_parts, tail_kb, tail_tiles;
    size_t rowg_off, scratch_off, partial_floats;      // float offsets into the partial area
    size_t strips_done_idx, tail_flags_idx, gen_idx, counters;
};

// units = work items (tiles or pair tiles), slots = CTAs or CTA pairs of the GPU, min_kb = fewest k-blocks a part is
// worth its hand-over with, fold_floats = row partials of the reduction (0: none), chain = the mean chain's per-row
// values follow them.
inline ScheduleLayout schedule_layout(int64_t tiles_m, int64_t tiles_n, int64_t units, int64_t slots, int num_kb, bool split_allowed,
                                      int min_kb, size_t fold_floats, bool chain, int64_t M)
{
    ScheduleLayout L = {};
    L.tiles_m = tiles_m;
    L.tiles_n = tiles_n;
    L.units = units;
    L.slots = slots;
    const int64_t full = units / slots, rest = units % slots;
    int parts = 1;
    if (split_allowed && rest > 0 && full < kTailMaxFullWaves) {
        int64_t s = slots / rest;
        if (s > kTailMaxParts) s = kTailMaxParts;
        if (s > num_kb / min_kb) s = num_kb / min_kb;
        parts = s < 1 ? 1 : (int)s;
    }
    L.tail_kb = (num_kb + parts - 1) / parts;
    L.tail_parts = (num_kb + L.tail_kb - 1) / L.tail_kb;       // no empty part
    L.tail_tiles = L.tail_parts > 1 ? (int)rest : 0;
    L.ctas = full > 0 ? slots : rest * L.tail_parts;
    L.rowg_off = fold_floats;                                  // mean chain: gelu(mean) per row after the partials
    L.scratch_off = (L.rowg_off + (chain ? (size_t)M : 0) + 3) / 4 * 4;
    // hand-over area: per cut tile, part, CTA of the pair and column half, 32 x 128 float4 of raw accumulators
    L.partial_floats = L.scratch_off + (size_t)L.tail_tiles * (L.tail_parts - 1) * 2 * 2 * (4 * 32 * kEpiGroupThreads);
    L.strips_done_idx = fold_floats ? (size_t)tiles_m : 0;
    L.tail_flags_idx = L.strips_done_idx + (chain ? 1 : 0);
    L.gen_idx = L.tail_flags_idx + (size_t)L.tail_tiles * 4;       // run index and finished-CTA count
    L.counters = L.gen_idx + 2;
    return L;
}

}  // namespace forge
