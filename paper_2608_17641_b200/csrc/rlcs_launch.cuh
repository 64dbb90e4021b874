// Host-side dispatch from (tile variant, truncation handling, vector alignment) to one
// instantiation of scan_kernel.  Each algorithm's translation unit instantiates its own kernels
// through RLCS_DEFINE_LAUNCHER so that the build can compile them in parallel.
#pragma once

#include "rlcs_scan.cuh"

namespace rlcs {

struct TileVariant { int threads, items, min_blocks; };
constexpr int kNumVariants = 4;
// variant 0 is the default; the others exist for the tiling-invariance tests and for tuning.
constexpr TileVariant kVariants[kNumVariants] = {
    {256, 8, 4},   // 2048 steps per tile
    {128, 4, 8},   //  512
    {512, 8, 2},   // 4096
    {256, 4, 4},   // 1024
};
constexpr int kMinTileElems = 512;

template <int ALGO, bool TRUNC, bool VEC, int V>
cudaError_t launch_variant(const ScanParams& p, cudaStream_t stream) {
    constexpr TileVariant tv = kVariants[V];
    scan_kernel<ALGO, TRUNC, VEC, tv.threads, tv.items, tv.min_blocks>
        <<<(unsigned)p.num_tiles, tv.threads, 0, stream>>>(p);
    return cudaGetLastError();
}

template <int ALGO, bool TRUNC, bool VEC>
cudaError_t launch_tv(const ScanParams& p, int variant, cudaStream_t stream) {
    switch (variant) {
        case 0: return launch_variant<ALGO, TRUNC, VEC, 0>(p, stream);
        case 1: return launch_variant<ALGO, TRUNC, VEC, 1>(p, stream);
        case 2: return launch_variant<ALGO, TRUNC, VEC, 2>(p, stream);
        case 3: return launch_variant<ALGO, TRUNC, VEC, 3>(p, stream);
        default: return cudaErrorInvalidValue;
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

#define RLCS_DEFINE_LAUNCHER(NAME, ALGO, HAS_TRUNC)                                                 \
    cudaError_t NAME(const ScanParams& p, int variant, bool trunc, bool vec, cudaStream_t stream) { \
        return launch_algo<ALGO, HAS_TRUNC>(p, variant, trunc, vec, stream);                        \
    }

}  // namespace rlcs
