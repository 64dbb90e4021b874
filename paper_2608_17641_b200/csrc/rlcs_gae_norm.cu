// GAE with advantage normalisation: the GAE scan kernel that also leaves per-tile sums, a one-block
// reduction of those sums to mean and 1/(std + eps), and the element-wise rescale of the advantages.
#include "rlcs_launch.cuh"

namespace rlcs {

RLCS_DEFINE_LAUNCHER(launch_gae_stats, kGaeStats, true)

// Sums of two doubles per thread over a block of 1024 threads, in a fixed order (lanes by shuffle
// distance 16, 8, ..., 1, then the 32 warp sums the same way in warp 0): every thread gets both.
__device__ __forceinline__ void block_sum2_1024(double& x, double& y, double* sh /* [66] */) {
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        x += __shfl_down_sync(0xffffffffu, x, d);
        y += __shfl_down_sync(0xffffffffu, y, d);
    }
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    if (lane == 0) { sh[w] = x; sh[32 + w] = y; }
    __syncthreads();
    if (w == 0) {
        double u = sh[lane], v = sh[32 + lane];
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) {
            u += __shfl_down_sync(0xffffffffu, u, d);
            v += __shfl_down_sync(0xffffffffu, v, d);
        }
        if (lane == 0) { sh[64] = u; sh[65] = v; }
    }
    __syncthreads();
    x = sh[64];
    y = sh[65];
}

// One block: per-tile {s_i = sum, q_i = sum of squared deviations from the tile mean} -> {mean,
// 1/(std + eps)}, in one strided pass in double followed by a block sum in a fixed order (the result
// does not depend on timing):
//     S = sum_i s_i,   Q = sum_i (q_i + s_i^2 / n_i),   sum (A - mean)^2 = Q - S^2 / N.
// The per-tile sums are fp32 and centred on the tile mean, so q_i carries no cancellation; s_i^2 is
// exact in double and the last subtraction loses 2^-52 (mean / std)^2 of relative accuracy -- 2e-10
// where the mean is a thousand standard deviations away.  Tile i of the scan order holds `tile` steps
// except the one at the array's end (scan-order tile 0 of this backward scan).
__global__ void __launch_bounds__(1024) norm_finalize_kernel(const float* __restrict__ partial, long long num_tiles,
                                                             long long total, int tile, int ddof, float eps,
                                                             float* __restrict__ out) {
    __shared__ double sh[66];
    grid_dependency_launch();
    grid_dependency_wait();                                  // the per-tile sums come from the kernel before
    const float2* const pairs = reinterpret_cast<const float2*>(partial);
    const long long last = total - (num_tiles - 1) * (long long)tile;      // steps in the ragged tile
    const double inv_tile = 1.0 / (double)tile, inv_last = 1.0 / (double)last;   // (no division per tile: one SM does all of this)
    double S = 0.0, Q = 0.0;
    for (long long i = threadIdx.x; i < num_tiles; i += 1024) {
        const float2 sq = __ldcg(pairs + i);
        const double si = (double)sq.x;
        S += si;
        Q += (double)sq.y + si * si * (i == 0 ? inv_last : inv_tile);
    }
    block_sum2_1024(S, Q, sh);
    if (threadIdx.x == 0) {
        const double mean = S / (double)total;
        const double ssd = fmax(Q - S * mean, 0.0);
        const double denom = (double)total - (double)ddof;
        const double var = denom > 0.0 ? ssd / denom : 0.0;
        out[0] = (float)mean;
        out[1] = (float)(1.0 / (sqrt(var) + (double)eps));
    }
}

// advantages <- (advantages - mean) * rstd, in place; 8 steps per thread with 256-bit accesses when
// the pointer allows, element-wise otherwise and for the ragged tail.
template <bool VEC>
__global__ void __launch_bounds__(256) norm_rescale_kernel(float* __restrict__ adv, long long total,
                                                           const float* mean_rstd) {
    grid_dependency_launch();
    grid_dependency_wait();                                  // mean and 1/(std + eps) come from the kernel before
    // plain loads: cached in L1 (every thread of the grid reads these two words -- bypassing L1 sends
    // them all to one L2 slice, measured +30 us), and issued only after the wait above
    const float mean = mean_rstd[0], rstd = mean_rstd[1];
    const long long i0 = ((long long)blockIdx.x * 256 + threadIdx.x) * 8;
    if (i0 >= total) return;
    if (VEC && i0 + 8 <= total) {
        float x[8];
        ldg_v8(adv + i0, x);
#pragma unroll
        for (int j = 0; j < 8; ++j) x[j] = (x[j] - mean) * rstd;
        stg_v8(adv + i0, x);
    } else {
        for (long long i = i0; i < total && i < i0 + 8; ++i) adv[i] = (adv[i] - mean) * rstd;
    }
}

// Both follow-up kernels are launched like the scan kernels: their blocks may be placed while the
// kernel before them drains, and they touch global memory only after grid_dependency_wait().
template <class Kernel, class... Args>
static cudaError_t launch_after(Kernel kernel, unsigned grid, unsigned block, cudaStream_t stream, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid, 1, 1);
    cfg.blockDim = dim3(block, 1, 1);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = rlcs_hooks::g_pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}

cudaError_t launch_norm_finalize(const float* partial, long long num_tiles, long long total, int tile, int ddof, float eps,
                                 float* mean_rstd, cudaStream_t stream) {
    return launch_after(norm_finalize_kernel, 1u, 1024u, stream, partial, num_tiles, total, tile, ddof, eps, mean_rstd);
}

cudaError_t launch_norm_rescale(float* adv, long long total, const float* mean_rstd, bool vec, cudaStream_t stream) {
    const long long blocks = (total + 2047) / 2048;
    const float* mr = mean_rstd;
    return vec ? launch_after(norm_rescale_kernel<true>, (unsigned)blocks, 256u, stream, adv, total, mr)
               : launch_after(norm_rescale_kernel<false>, (unsigned)blocks, 256u, stream, adv, total, mr);
}

}  // namespace rlcs
