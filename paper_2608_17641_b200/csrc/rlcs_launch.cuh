// Host-side dispatch from (tile variant, truncation handling, pointer alignment) to one
// instantiation of the scan kernels.  Each algorithm's translation unit instantiates its own
// kernels through RLCS_DEFINE_LAUNCHER so that the build can compile them in parallel.
#pragma once

#include "rlcs_scan.cuh"

namespace rlcs_hooks {
extern bool g_pdl;                 // launch with programmatic stream serialisation (default on)
}

namespace RLCS_NS {

// Every scan kernel goes through this launch: grid/block/shared memory, an optional thread-block
// cluster size, and programmatic stream serialisation, which lets the blocks of this launch be
// placed while the previous kernel of the stream drains (the kernels call grid_dependency_wait()
// before they touch global memory, so ordering on the stream is unchanged).
template <class Kernel>
cudaError_t launch_scan(Kernel kernel, unsigned grid, unsigned block, size_t smem, cudaStream_t stream, int cluster,
                        const ScanParams& p) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid, 1, 1);
    cfg.blockDim = dim3(block, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    unsigned n = 0;
    if (cluster > 1) {
        attr[n].id = cudaLaunchAttributeClusterDimension;
        attr[n].val.clusterDim.x = (unsigned)cluster;
        attr[n].val.clusterDim.y = 1;
        attr[n].val.clusterDim.z = 1;
        ++n;
    }
    if (rlcs_hooks::g_pdl) {
        attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n].val.programmaticStreamSerializationAllowed = 1;
        ++n;
    }
    cfg.attrs = attr;
    cfg.numAttrs = n;
    return cudaLaunchKernelEx(&cfg, kernel, p);
}

// stages == 0: scan_kernel (one tile per block).  stages > 0: scan_kernel_tma (persistent blocks,
// bulk-copy ring of that many tiles; min_blocks = blocks per SM it is compiled and sized for).
struct TileVariant { int threads, items, min_blocks, stages; };
constexpr int kNumVariants = 22;
constexpr TileVariant kVariants[kNumVariants] = {
    {256, 8, 4, 0},    //  0: 2048 steps per tile
    {128, 4, 8, 0},    //  1:  512
    {512, 8, 2, 0},    //  2: 4096
    {256, 4, 4, 0},    //  3: 1024
    {256, 16, 2, 0},   //  4: 4096
    {128, 16, 4, 0},   //  5: 2048
    {128, 8, 8, 0},    //  6: 1024
    {512, 16, 1, 0},   //  7: 8192
    {256, 8, 3, 3},    //  8: 2048, persistent, 3 stages
    {256, 8, 2, 4},    //  9: 2048, persistent, 4 stages
    {256, 8, 4, 2},    // 10: 2048, persistent, 2 stages
    {128, 8, 6, 3},    // 11: 1024, persistent, 3 stages
    {512, 8, 1, 3},    // 12: 4096, persistent, 3 stages
    {256, 16, 2, 2},   // 13: 4096, persistent, 2 stages
    {256, 8, 3, 4},    // 14: 2048, persistent, 4 stages
    {256, 8, 3, 6},    // 15: 2048, persistent, 6 stages
    {256, 8, 5, 0},    // 16: 2048, at most 48 registers
    {256, 8, 6, 0},    // 17: 2048, at most 40 registers
    {128, 16, 5, 0},   // 18: 2048, 16 steps per thread
    {128, 16, 6, 0},   // 19: 2048, 16 steps per thread, at most 80 registers
    {128, 16, 8, 0},   // 20: 2048, 16 steps per thread, at most 64 registers
    {128, 16, 10, 0},  // 21: 2048, 16 steps per thread, at most 48 registers (bfloat16 build only)
};
// Which rows of the table are compiled.  The default build holds the shapes the selection in
// choose_variant() can return (0, 1, 5, 6, 18, 19, 20) and two persistent bulk-copy ring shapes (8, 11)
// that the tests cross-check against; the rest of the table is tuning history and is compiled only
// with -DRLCS_ALL_VARIANTS.  The bfloat16 build instantiates 16-steps-per-thread shapes (one 32-byte
// access) and the two 8-step ones; the observation-skip scans and the bare affine scan (a test
// hook) fewer still.
#ifdef RLCS_ALL_VARIANTS
constexpr bool kAllVariants = true;
#else
constexpr bool kAllVariants = false;
#endif
__host__ __device__ constexpr bool variant_built(int v) {
    if (kIoBf16) return v == 0 || v == 5 || v == 6 || v >= 18;
    return kAllVariants || v == 0 || v == 1 || v == 5 || v == 6 || v == 8 || v == 11 || (v >= 18 && v <= 20);
}
__host__ __device__ constexpr bool variant_built_for(int algo, int v) {
    if (!variant_built(v)) return false;
    if (uses_skip(algo)) return v == 0 || v == 6 || v >= 18;
    if (is_affine(algo)) return kAllVariants || v == 0 || v == 6;
    if (algo == kGaeStats) return kAllVariants || v == 0 || v == 1 || v == 6 || v == 19;
    return true;
}
constexpr int kMinTileElems = 512;
constexpr int kRetraceProbsThreads = 256, kRetraceProbsItems = 4;      // tile of rlcs_retrace_probs
constexpr int kMaxDevices = 64;

template <int ALGO, bool TRUNC, int V>
cudaError_t launch_persistent(const ScanParams& p, cudaStream_t stream) {
    constexpr TileVariant tv = kVariants[V];
    constexpr int STAGES = tv.stages > 0 ? tv.stages : 1;
    using L = StageLayout<ALGO, TRUNC, tv.threads * tv.items>;
    constexpr size_t kSmem = (size_t)STAGES * L::BYTES;
    auto kernel = scan_kernel_tma<ALGO, TRUNC, tv.threads, tv.items, STAGES, tv.min_blocks>;
    // Per-device launch configuration, found once: the grid must not exceed what is co-resident,
    // because a block may wait for the tile record of any block with a smaller index.
    static int s_blocks[kMaxDevices] = {};
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    if (s_blocks[dev] == 0) {
        err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmem);
        if (err != cudaSuccess) return err;
        int per_sm = 0, sms = 0;
        err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, tv.threads, kSmem);
        if (err != cudaSuccess) return err;
        err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (err != cudaSuccess) return err;
        if (per_sm < 1 || sms < 1) return cudaErrorLaunchOutOfResources;
        s_blocks[dev] = per_sm * sms;
    }
    const long long grid = p.num_tiles < s_blocks[dev] ? p.num_tiles : s_blocks[dev];
    return launch_scan(kernel, (unsigned)grid, tv.threads, kSmem, stream, 0, p);
}

// One cluster per row (p.cluster = tiles per row, 2..8): carry through distributed shared memory.
template <int ALGO, bool TRUNC, int V>
cudaError_t launch_cluster(const ScanParams& p, cudaStream_t stream) {
    constexpr TileVariant tv = kVariants[V];
    return launch_scan(scan_kernel_cluster<ALGO, TRUNC, tv.threads, tv.items, tv.min_blocks>, (unsigned)p.num_tiles, tv.threads, 0,
                       stream, p.cluster, p);
}

// One thread block per row (p.row_blocks; rows longer than a tile, many rows): grid = number of rows.
template <int ALGO, bool TRUNC, int V>
cudaError_t launch_rows(const ScanParams& p, cudaStream_t stream) {
    constexpr TileVariant tv = kVariants[V];
    return launch_scan(scan_kernel_rows<ALGO, TRUNC, tv.threads, tv.items, tv.min_blocks>, (unsigned)p.num_tiles, tv.threads, 0,
                       stream, 0, p);
}

// algorithms that have the one-block-per-row kernel (the seven of the paper, the bare affine scan, and
// GAE with per-tile statistics -- for rows of whole tiles, which the host checks)
__host__ __device__ constexpr bool has_row_blocks(int algo) { return algo <= kAffineFwd || algo == kGaeStats; }
// algorithms that have the row-aligned tiling instantiation of the one-tile kernel
__host__ __device__ constexpr bool has_row_tiles(int algo) { return algo <= kAffineFwd; }

template <int ALGO, bool TRUNC, bool VEC, int V>
cudaError_t launch_variant(const ScanParams& p, cudaStream_t stream) {
    constexpr TileVariant tv = kVariants[V];
    if constexpr (VEC && tv.stages == 0 && has_row_blocks(ALGO)) {
        if (p.row_blocks) return launch_rows<ALGO, TRUNC, V>(p, stream);
    }
    if constexpr (VEC && tv.stages == 0) {
        if (p.cluster > 1) return launch_cluster<ALGO, TRUNC, V>(p, stream);
    }
    if constexpr (tv.stages > 0 && VEC) {
        // (rows shorter than a chunk go to the one-tile kernel: the persistent one assumes T >= ITEMS)
        if (p.T >= (unsigned)tv.items) return launch_persistent<ALGO, TRUNC, V>(p, stream);
        return launch_scan(scan_kernel<ALGO, TRUNC, true, tv.threads, tv.items, tv.min_blocks>, (unsigned)p.num_tiles, tv.threads,
                           0, stream, 0, p);
    } else {
        if constexpr (has_row_tiles(ALGO)) {
            // row-aligned tiling has an instantiation of its own (idle tail threads, tile length at run time)
            if (p.tile_steps != (unsigned)(tv.threads * tv.items))
                return launch_scan(scan_kernel<ALGO, TRUNC, VEC, tv.threads, tv.items, tv.min_blocks, true>, (unsigned)p.num_tiles,
                                   tv.threads, 0, stream, 0, p);
        }
        // bulk copies need 16-byte aligned pointers; otherwise the element-wise kernel of the same tile shape
        return launch_scan(scan_kernel<ALGO, TRUNC, VEC, tv.threads, tv.items, tv.min_blocks>, (unsigned)p.num_tiles, tv.threads,
                           0, stream, 0, p);
    }
}

template <int ALGO, bool TRUNC, bool VEC, int V = 0>
cudaError_t launch_tv(const ScanParams& p, int variant, cudaStream_t stream) {
    if constexpr (V >= kNumVariants) {
        return cudaErrorInvalidValue;
    } else {
        if constexpr (variant_built_for(ALGO, V)) {
            if (variant == V) return launch_variant<ALGO, TRUNC, VEC, V>(p, stream);
        }
        return launch_tv<ALGO, TRUNC, VEC, V + 1>(p, variant, stream);
    }
}

template <int ALGO, bool HAS_TRUNC_VARIANT>
cudaError_t launch_algo(const ScanParams& p, int variant, bool trunc, bool vec, cudaStream_t stream) {
    if constexpr (HAS_TRUNC_VARIANT) {
        if (trunc) return vec ? launch_tv<ALGO, true, true>(p, variant, stream)
                              : launch_tv<ALGO, true, false>(p, variant, stream);
    }
    return vec ? launch_tv<ALGO, false, true>(p, variant, stream)
               : launch_tv<ALGO, false, false>(p, variant, stream);
}

// One launcher per algorithm, defined in that algorithm's .cu file.
cudaError_t launch_gae(const ScanParams&, int variant, bool trunc, bool vec, cudaStream_t);
cudaError_t launch_td_lambda(const ScanParams&, int variant, bool trunc, bool vec, cudaStream_t);
cudaError_t launch_disc(const ScanParams&, int variant, bool trunc, bool vec, cudaStream_t);
cudaError_t launch_vtrace(const ScanParams&, int variant, bool trunc, bool vec, cudaStream_t);
cudaError_t launch_retrace(const ScanParams&, int variant, bool trunc, bool vec, cudaStream_t);
cudaError_t launch_elig(const ScanParams&, int variant, bool trunc, bool vec, cudaStream_t);
cudaError_t launch_prefix(const ScanParams&, int variant, bool trunc, bool vec, cudaStream_t);
cudaError_t launch_affine_bwd(const ScanParams&, int variant, bool trunc, bool vec, cudaStream_t);
cudaError_t launch_affine_fwd(const ScanParams&, int variant, bool trunc, bool vec, cudaStream_t);
cudaError_t launch_retrace_probs(const ScanParams&, bool trunc, bool vec, bool vec_rows, cudaStream_t);
cudaError_t launch_gae_stats(const ScanParams&, int variant, bool trunc, bool vec, cudaStream_t);
cudaError_t launch_gae_skip(const ScanParams&, int variant, bool trunc, bool vec, cudaStream_t);
cudaError_t launch_norm_finalize(const float* partial, long long num_tiles, long long total, int tile, int ddof, float eps,
                                 float* mean_rstd, cudaStream_t stream);
cudaError_t launch_norm_rescale(float* adv, long long total, const float* mean_rstd, bool vec, cudaStream_t stream);

#define RLCS_DEFINE_LAUNCHER(NAME, ALGO, HAS_TRUNC)                                                 \
    cudaError_t NAME(const ScanParams& p, int variant, bool trunc, bool vec, cudaStream_t stream) { \
        return launch_algo<ALGO, HAS_TRUNC>(p, variant, trunc, vec, stream);                        \
    }

}  // namespace RLCS_NS
