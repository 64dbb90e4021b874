// Kernel instantiations for GAE with observation-skip masking: the fused kernel that runs the value
// fill and the masked GAE scan in one pass over each tile (see rlcs_scan.cuh).
#include "rlcs_launch.cuh"

namespace rlcs {

template <bool TRUNC, bool VEC, int V>
cudaError_t launch_skip_variant(const ScanParams& p, cudaStream_t stream) {
    constexpr TileVariant tv = kVariants[V];
    if constexpr (VEC) {
        // rows of whole tiles and many of them: one thread block per row, both carries in registers
        if (p.row_blocks)
            return launch_scan(scan_kernel_gae_skip_rows<TRUNC, tv.threads, tv.items, tv.min_blocks>, (unsigned)p.num_tiles,
                               tv.threads, 0, stream, 0, p);
    }
    return launch_scan(scan_kernel_gae_skip<TRUNC, VEC, tv.threads, tv.items, tv.min_blocks>, (unsigned)p.num_tiles, tv.threads, 0,
                       stream, 0, p);
}

template <bool TRUNC, bool VEC>
cudaError_t launch_skip_tv(const ScanParams& p, int variant, cudaStream_t stream) {
    switch (variant) {                       // the tile shapes variant_built_for() lists for these scans
        case 0: return launch_skip_variant<TRUNC, VEC, 0>(p, stream);
        case 6: return launch_skip_variant<TRUNC, VEC, 6>(p, stream);
        case 18: return launch_skip_variant<TRUNC, VEC, 18>(p, stream);
        case 19: return launch_skip_variant<TRUNC, VEC, 19>(p, stream);
        case 20: return launch_skip_variant<TRUNC, VEC, 20>(p, stream);
        default: return cudaErrorInvalidValue;
    }
}

cudaError_t launch_gae_skip(const ScanParams& p, int variant, bool trunc, bool vec, cudaStream_t stream) {
    if (trunc) return vec ? launch_skip_tv<true, true>(p, variant, stream) : launch_skip_tv<true, false>(p, variant, stream);
    return vec ? launch_skip_tv<false, true>(p, variant, stream) : launch_skip_tv<false, false>(p, variant, stream);
}

}  // namespace rlcs
