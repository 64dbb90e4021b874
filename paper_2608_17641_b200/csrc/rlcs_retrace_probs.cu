// Retrace(lambda) from [N,T,A] Q-values and action probabilities: kernel instantiations.
// One tile shape (256 threads x 4 steps: the per-step work is A-wide already), A = 4 / 8 / 16
// specialised with vector loads, any other A through the generic loop.
#include "rlcs_launch.cuh"

namespace rlcs {

template <bool TRUNC, bool VEC, int AV>
static cudaError_t launch_one(const ScanParams& p, cudaStream_t stream) {
    if constexpr (VEC) {
        // rows of whole tiles and many of them: one thread block per row, the carry in a register
        if (p.row_blocks)
            return launch_scan(scan_kernel_retrace_probs_rows<TRUNC, kRetraceProbsThreads, kRetraceProbsItems, 4, AV>,
                               (unsigned)p.num_tiles, kRetraceProbsThreads, 0, stream, 0, p);
    }
    return launch_scan(scan_kernel_retrace_probs<TRUNC, VEC, kRetraceProbsThreads, kRetraceProbsItems, 4, AV>,
                       (unsigned)p.num_tiles, kRetraceProbsThreads, 0, stream, 0, p);
}

template <bool TRUNC, bool VEC>
static cudaError_t launch_a(const ScanParams& p, bool vec_rows, cudaStream_t stream) {
    // 256-bit loads of the [.,A] rows need 32-byte aligned Q / pi / mu pointers and A = 4, 8 or 16
    if (vec_rows && p.A == 4) return launch_one<TRUNC, VEC, 4>(p, stream);
    if (vec_rows && p.A == 8) return launch_one<TRUNC, VEC, 8>(p, stream);
    if (vec_rows && p.A == 16) return launch_one<TRUNC, VEC, 16>(p, stream);
    return launch_one<TRUNC, VEC, 0>(p, stream);
}

cudaError_t launch_retrace_probs(const ScanParams& p, bool trunc, bool vec, bool vec_rows, cudaStream_t stream) {
    if (trunc) return vec ? launch_a<true, true>(p, vec_rows, stream) : launch_a<true, false>(p, vec_rows, stream);
    return vec ? launch_a<false, true>(p, vec_rows, stream) : launch_a<false, false>(p, vec_rows, stream);
}

}  // namespace rlcs
