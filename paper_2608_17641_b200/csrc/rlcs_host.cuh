// Host-side helpers shared by the fp32 and bfloat16 C-ABI translation units: argument validation,
// kernel selection, tiling and workspace wiring.  Included after rlcs_launch.cuh; everything here
// refers to the build's own namespace (RLCS_NS) and element type (io_t).
#pragma once

#include <cmath>
#include <cstdint>

#include "../../include/rlcs.h"
#include "rlcs_device.cuh"
#include "rlcs_launch.cuh"

// test hooks, set through the rlcs_debug_* entry points (defined in rlcs_api.cu)
namespace rlcs_hooks {
extern int g_variant;              // tile variant; -1 = chosen per call by choose_variant
extern bool g_cluster;             // allow the cluster carry
extern bool g_wide_index;          // use the 64-bit index path even when 32 bits would do
extern long long g_mute_tile;      // tile that does not publish
extern long long g_spin_cap;       // poll limit (0 = default)
extern bool g_row_tiles;           // allow row-aligned tiling (default on)
extern int g_row_blocks;           // one thread block per row: -1 = when there are enough rows (default), 0 = never, 1 = whenever legal
}  // namespace rlcs_hooks

namespace {

using RLCS_NS::ScanParams;
using RLCS_NS::io_t;
using rlcs_hooks::g_variant;
using rlcs_hooks::g_cluster;
using rlcs_hooks::g_wide_index;
using rlcs_hooks::g_mute_tile;
using rlcs_hooks::g_spin_cap;
constexpr unsigned kDefaultSpinCap = 1u << 21;

constexpr int64_t kMaxT = (int64_t(1) << 31) - 1;
constexpr int64_t kMaxTotal = int64_t(1) << 40;

inline bool aligned(const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }
inline bool unit_interval(float v) { return v >= 0.f && v <= 1.f; }   // false for NaN
inline bool clip_ok(float v) { return v >= 0.f; }                       // false for NaN; +inf allowed

int tile_elems(int variant) { return RLCS_NS::kVariants[variant].threads * RLCS_NS::kVariants[variant].items; }

// size check common to every entry point; returns RLCS_OK with *total = 0 for empty problems
int check_sizes(int64_t N, int64_t T, int64_t* total) {
    *total = 0;
    if (N < 0 || T < 0 || T > kMaxT) return RLCS_ERR_SIZE;
    if (N == 0 || T == 0) return RLCS_OK;
    if (N > kMaxTotal / T) return RLCS_ERR_SIZE;
    *total = N * T;
    return RLCS_OK;
}

struct Ptrs {
    const void* f32[8];
    int nf32 = 0;
    const void* u8[2];
    int nu8 = 0;
    void add_f32(const void* p) { if (p) f32[nf32++] = p; }
    void add_u8(const void* p) { if (p) u8[nu8++] = p; }
};

// RLCS_ERR_ALIGN if a float-tensor pointer is not aligned to its element; *vec = all pointers allow vector access
int check_alignment(const Ptrs& ps, bool* vec) {
    *vec = true;
    for (int i = 0; i < ps.nf32; ++i) {
        if (!aligned(ps.f32[i], sizeof(io_t))) return RLCS_ERR_ALIGN;
        if (!aligned(ps.f32[i], 32)) *vec = false;          // 256-bit vector accesses
    }
    for (int i = 0; i < ps.nu8; ++i)
        if (!aligned(ps.u8[i], 16)) *vec = false;
    return RLCS_OK;
}

// Kernel and tile shape for one call, from measurements on B200 (see the tile-variant table in
// rlcs_launch.cuh).  Large problems are bound by HBM: what matters is resident warps and bytes in
// flight, so algorithms with few registers run more blocks per SM or 16 steps per thread.  Small
// problems are bound by latency: smaller tiles spread them over more SMs, unless rows are long
// enough for the inter-block carry to dominate.
int choose_variant_unchecked(int algo, bool trunc, int64_t total, int64_t T) {
    if (total < (int64_t(1) << 23)) {
        // latency-bound sizes (cold-L2 sweeps): long rows want few carry hops (2048-step tiles, one
        // cluster per row where that fits), the smallest problems want many small blocks
        // (the 16-step shape at 80 registers spills for the algorithms with three or four float inputs:
        // V-trace takes it at 96 registers, Retrace the 8-step shape of the same tile length)
        if (T > 2048) return algo == RLCS_NS::kRetrace ? 0 : algo == RLCS_NS::kVtrace ? 18 : 19;
        return total <= (int64_t(1) << 19) ? 1 : 6;
    }
    if (RLCS_NS::kIoBf16) {
        // 16 steps per thread (one 32-byte access per tensor).  With half the bytes per step the kernels
        // are bound by issue slots and latency, and resident blocks pay even with a few spills: every
        // algorithm with truncation handling runs fastest at 8 blocks per SM (measured over all built
        // shapes at 16384 x 2048: Retrace 0.82 -> 0.90, V-trace 0.75 -> 0.77 against 6 blocks), and the
        // three lightest kernels at 10 (discounted return 0.70 -> 0.74, forward scans 0.81 -> 0.84).
        if (algo == RLCS_NS::kDisc || algo == RLCS_NS::kElig || algo == RLCS_NS::kPrefix) return 21;
        return trunc ? 20 : 18;
    }
    switch (algo) {
        case RLCS_NS::kGae: return trunc ? 19 : 0;
        case RLCS_NS::kGaeStats: return trunc ? 19 : 0;
        case RLCS_NS::kVtrace: return trunc ? 18 : 0;
        case RLCS_NS::kRetrace: return 0;
        case RLCS_NS::kTdLambda: return trunc ? 20 : 0;
        case RLCS_NS::kDisc: return trunc ? 20 : 5;
        case RLCS_NS::kFillSkip:
        case RLCS_NS::kGaeSkip: return 18;
        case RLCS_NS::kElig: return 18;
        case RLCS_NS::kPrefix: return 18;
        default: return 0;
    }
}

// A row longer than the variant's tile splits into whole chunks and fills its tiles to at least 70 %:
// what the one-thread-block-per-row kernel needs of (variant, T).
bool row_fits(int variant, int64_t T) {
    const RLCS_NS::TileVariant tv = RLCS_NS::kVariants[variant];
    const int64_t tile = (int64_t)tv.threads * tv.items;
    if (tv.stages != 0 || T <= tile || T % tv.items != 0) return false;
    const int64_t tiles = (T + tile - 1) / tile;
    return T * 10 >= tiles * tile * 7;
}

// Rows a little more numerous than the thread blocks the GPU holds at once (up to 1.2 times): with one
// block per row the few blocks of the second wave finish the call alone, one per SM (measured, GAE
// 900 x 16384: 0.72 of the copy bandwidth against 0.78 with the cluster carry; 1024 x 32768: 0.78 either
// way; 1200 x 16384: 0.82 against 0.81).
bool thin_second_wave(int variant, int64_t rows) {
    const int64_t slots = (int64_t)rlcs_device::limits().sms * RLCS_NS::kVariants[variant].min_blocks;
    return rows > slots && rows * 5 < slots * 6;
}

int choose_variant(int algo, bool trunc, int64_t total, int64_t T) {
    if (g_variant >= 0 && RLCS_NS::variant_built_for(algo, g_variant)) return g_variant;
    int v = choose_variant_unchecked(algo, trunc, total, T);
    // Long rows, enough of them for one thread block per row: if the preferred shape does not suit the
    // row length (T not a multiple of its 16 steps per thread, or a mostly empty last tile), an 8-step
    // shape that does is worth more than the preferred shape with a carry between blocks.
    if (rlcs_hooks::g_row_blocks != 0 && RLCS_NS::variant_built_for(algo, v) && T > tile_elems(v) &&
        total / T >= 3 * rlcs_device::limits().sms && !row_fits(v, T)) {
        const int alternatives[2] = {0, 6};          // 256 x 8 (2048 steps), 128 x 8 (1024 steps)
        for (int alt : alternatives)
            if (RLCS_NS::variant_built_for(algo, alt) && row_fits(alt, T) && !thin_second_wave(alt, total / T)) { v = alt; break; }
    }
    if (RLCS_NS::variant_built_for(algo, v)) return v;
    // not compiled for this algorithm / element type: the nearest shape that every build has
    return (total < (int64_t(1) << 23) && T <= 2048) ? 6 : 0;
}

// How the carry between thread blocks travels for one call, and the workspace bytes it needs.
struct CarryPlan {
    int carry_mode;      // rows straddle tiles: tile records in the workspace, look-back
    int cluster;         // > 1: one thread-block cluster of this many tiles per row, no workspace
    size_t bytes;        // workspace bytes this call reads or writes (0 when it needs none)
    int tile_steps;      // steps per thread block: the tile, or less with row-aligned tiling
    int row_blocks;      // one thread block per row, walking the row's tiles (no carry between blocks)
};

// Row-aligned tiling: when rows are shorter than a tile but do not divide it, a block can take the
// largest whole number of rows that fits (k*T steps) instead of a full tile, provided every thread
// still gets either a whole chunk or nothing (k*T a multiple of the steps per thread) and few
// threads idle (at least 70 % of the tile used).  No row straddles a tile then, so there is no
// carry between blocks at all: no workspace traffic, no waiting on other blocks.  T = 1000 on
// 1024-step tiles idles 3 threads of 128; T = 2000, 500, 250, 200, 100 fit 2048-step tiles the same way.
int row_aligned_steps(int variant, int64_t T) {
    const int tile = tile_elems(variant), items = RLCS_NS::kVariants[variant].items;
    if (!rlcs_hooks::g_row_tiles || RLCS_NS::kVariants[variant].stages != 0 || T > tile || tile % T == 0) return 0;
    if (T < items) return 0;
    for (int64_t rows = tile / T; rows * T * 10 >= (int64_t)tile * 7; --rows)      // fewer rows if the most that fit do not split into whole chunks
        if ((rows * T) % items == 0) return (int)(rows * T);
    return 0;
}

// One thread block per row: rows longer than a tile, T a multiple of the steps per thread (every
// chunk whole and aligned), vector access, the row's tiles at least 70 % used, and at least three
// rows per SM (with fewer rows too many SMs idle: those go to the cluster carry or the look-back;
// measured cross-over at T = 16384: 384 rows 0.70 against 0.73, 512 rows 0.84 against 0.70).
bool row_blocks_ok(int variant, int64_t total, int64_t T, bool vec, bool any_wave = false) {
    const RLCS_NS::TileVariant tv = RLCS_NS::kVariants[variant];
    const int tile = tv.threads * tv.items;
    if (rlcs_hooks::g_row_blocks == 0 || !vec || tv.stages != 0 || T <= tile || T % tv.items != 0) return false;
    const int64_t tiles = (T + tile - 1) / tile;
    if (T * 10 < tiles * tile * 7) return false;
    if (rlcs_hooks::g_row_blocks > 0) return true;
    if (!any_wave && thin_second_wave(variant, total / T)) return false;
    return total / T >= 3 * rlcs_device::limits().sms;        // measured cross-over against the cluster carry: about 3 rows per SM
}

// allow_row_blocks: 0 = never, 1 = where row_blocks_ok() says so, 2 = the same without its rule about a thin
// second wave (for kernels whose carry between blocks costs more than such a wave does).
CarryPlan plan_carry(int variant, int64_t total, int64_t T, bool vec, bool allow_cluster, int records_per_tile,
                     bool allow_row_tiles = true, int allow_row_blocks = 1) {
    const int tile = tile_elems(variant);
    const int64_t num_tiles = (total + tile - 1) / tile;
    CarryPlan plan = {(tile % T) != 0 ? 1 : 0, 0, 0, tile, 0};    // T does not divide the tile: rows straddle tiles
    if (allow_row_blocks && row_blocks_ok(variant, total, T, vec, allow_row_blocks == 2)) {
        plan.carry_mode = 0;
        plan.row_blocks = 1;
        return plan;
    }
    if (plan.carry_mode && allow_row_tiles) {
        const int steps = row_aligned_steps(variant, T);
        if (steps > 0) {
            plan.carry_mode = 0;
            plan.tile_steps = steps;
            return plan;
        }
    }
    // Rows of exactly 2..8 tiles: one thread-block cluster per row carries through distributed
    // shared memory instead (needs the vectorised one-tile kernel; g_cluster = 0 turns it off).
    if (allow_cluster && g_cluster && vec && RLCS_NS::kVariants[variant].stages == 0 && T % tile == 0 && T / tile >= 2 &&
        T / tile <= 8) {
        plan.cluster = (int)(T / tile);
        plan.carry_mode = 0;
    }
    if (plan.carry_mode)
        plan.bytes = sizeof(unsigned) * RLCS_NS::kHeaderWords + sizeof(uint4) * (size_t)num_tiles * records_per_tile;
    return plan;
}

// Fill the size / tiling / carry fields and validate the workspace for this call.  Callers whose
// kernels have no row-aligned / one-block-per-row instantiation (has_row_blocks() in rlcs_launch.cuh:
// the statistics flavour of GAE, the observation-skip scans) pass allow_row_tiles = allow_row_blocks =
// false; Retrace from [N,T,A] tensors has its own one-block-per-row kernel for rows of whole tiles.
int finish_params(ScanParams& p, int variant, int64_t total, int64_t T, void* workspace, size_t workspace_bytes, bool vec,
                  bool allow_cluster = true, int records_per_tile = 1, bool allow_row_tiles = true, int allow_row_blocks = 1) {
    const int tile = tile_elems(variant);
    const CarryPlan plan = plan_carry(variant, total, T, vec, allow_cluster, records_per_tile, allow_row_tiles, allow_row_blocks);
    p.total = total;
    p.T = (unsigned)T;
    p.tile_steps = (unsigned)plan.tile_steps;
    p.num_tiles = plan.row_blocks ? total / T : (total + plan.tile_steps - 1) / plan.tile_steps;      // = the grid
    p.row_blocks = plan.row_blocks;
    p.idx32 = !g_wide_index && (total + tile) <= 0xffffffffLL;
    {   // invariant division by T (see FastDiv)
        int l = 0;
        while ((int64_t(1) << l) < T) ++l;
        p.div_T.mul = (unsigned)((((uint64_t(1) << 32) * ((uint64_t(1) << l) - (uint64_t)T)) / (uint64_t)T) + 1);
        p.div_T.sh1 = l < 1 ? l : 1;
        p.div_T.sh2 = l > 1 ? l - 1 : 0;
    }
    p.decay_pow = 1.f;                       // beta product of a chunk without resets
    for (int i = 0; i < RLCS_NS::kVariants[variant].items; ++i) p.decay_pow *= p.decay;
    p.carry_mode = plan.carry_mode;
    p.cluster = plan.cluster;
    p.header = nullptr;
    p.records = nullptr;
    p.status = nullptr;
    if (workspace != nullptr && workspace_bytes >= sizeof(unsigned) * RLCS_NS::kHeaderWords && aligned(workspace, 16))
        p.status = static_cast<unsigned*>(workspace) + 2;
    p.mute_tile = g_mute_tile;
    p.spin_cap = g_spin_cap > 0 ? (unsigned)g_spin_cap : kDefaultSpinCap;
    if (p.carry_mode) {
        if (workspace == nullptr || workspace_bytes < plan.bytes) return RLCS_ERR_WORKSPACE;
        if (!aligned(workspace, 16)) return RLCS_ERR_ALIGN;
        p.header = static_cast<unsigned*>(workspace);
        p.records = reinterpret_cast<uint4*>(p.header + RLCS_NS::kHeaderWords);
    }
    return RLCS_OK;
}

typedef cudaError_t (*Launcher)(const ScanParams&, int, bool, bool, cudaStream_t);

int run(Launcher fn, const ScanParams& p, int variant, bool trunc, bool vec, void* stream) {
    return fn(p, variant, trunc, vec, static_cast<cudaStream_t>(stream)) == cudaSuccess ? RLCS_OK : RLCS_ERR_CUDA;
}

// shared front half of the five backward entry points
int backward_common(ScanParams& p, Ptrs& ps, const uint8_t* dones, const uint8_t* truncs,
                    const io_t* trunc_bootstrap, const io_t* bootstrap, int64_t N, int64_t T,
                    int64_t* total, bool* vec) {
    int st = check_sizes(N, T, total);
    if (st != RLCS_OK || *total == 0) return st;
    if (dones == nullptr || (truncs == nullptr) != (trunc_bootstrap == nullptr)) return RLCS_ERR_NULL;
    ps.add_u8(dones);
    ps.add_u8(truncs);
    ps.add_f32(trunc_bootstrap);
    ps.add_f32(bootstrap);
    st = check_alignment(ps, vec);
    if (st != RLCS_OK) return st;
    p.dones = dones;
    p.truncs = truncs;
    p.trunc_boot = trunc_bootstrap;
    p.boot = bootstrap;
    return RLCS_OK;
}

}  // namespace
