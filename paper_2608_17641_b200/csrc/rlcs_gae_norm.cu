// GAE with advantage normalisation: the GAE scan kernel that also leaves per-tile sums, a one-block
// reduction of those sums to mean and 1/(std + eps), and the element-wise rescale of the advantages.
#include "rlcs_launch.cuh"

namespace rlcs {

RLCS_DEFINE_LAUNCHER(launch_gae_stats, kGaeStats, true)

// One block: per-tile {sum, sum of squared deviations from the tile mean} -> {mean, 1/(std + eps)}.
// Two strided passes in double, each followed by a shared-memory tree in a fixed order (the result
// does not depend on timing): first the mean, then
//     sum (A - mean)^2 = sum over tiles of [ q_i + n_i (m_i - mean)^2 ],   m_i = s_i / n_i,
// which is exact algebra and never subtracts two large numbers.  Tile i of the scan order holds
// `tile` steps except the one at the array's end (scan-order tile 0 of this backward scan).
__global__ void __launch_bounds__(1024) norm_finalize_kernel(const float* __restrict__ partial, long long num_tiles,
                                                             long long total, int tile, int ddof, float eps,
                                                             float* __restrict__ out) {
    __shared__ double sh[1024];
    __shared__ double mean_sh;
    double acc = 0.0;
    for (long long i = threadIdx.x; i < num_tiles; i += 1024) acc += (double)partial[2 * i];
    sh[threadIdx.x] = acc;
    __syncthreads();
    for (int d = 512; d > 0; d >>= 1) {
        if ((int)threadIdx.x < d) sh[threadIdx.x] += sh[threadIdx.x + d];
        __syncthreads();
    }
    if (threadIdx.x == 0) mean_sh = sh[0] / (double)total;
    __syncthreads();
    const double mean = mean_sh;
    const long long last = total - (num_tiles - 1) * (long long)tile;      // steps in the ragged tile
    acc = 0.0;
    for (long long i = threadIdx.x; i < num_tiles; i += 1024) {
        const double n = (double)(i == 0 ? last : (long long)tile);
        const double dm = (double)partial[2 * i] / n - mean;
        acc += (double)partial[2 * i + 1] + n * dm * dm;
    }
    sh[threadIdx.x] = acc;
    __syncthreads();
    for (int d = 512; d > 0; d >>= 1) {
        if ((int)threadIdx.x < d) sh[threadIdx.x] += sh[threadIdx.x + d];
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        const double denom = (double)total - (double)ddof;
        const double var = denom > 0.0 ? sh[0] / denom : 0.0;
        out[0] = (float)mean;
        out[1] = (float)(1.0 / (sqrt(var) + (double)eps));
    }
}

// advantages <- (advantages - mean) * rstd, in place; 8 steps per thread with 256-bit accesses when
// the pointer allows, element-wise otherwise and for the ragged tail.
template <bool VEC>
__global__ void __launch_bounds__(256) norm_rescale_kernel(float* __restrict__ adv, long long total,
                                                           const float* __restrict__ mean_rstd) {
    const float mean = __ldg(mean_rstd), rstd = __ldg(mean_rstd + 1);
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

cudaError_t launch_norm_finalize(const float* partial, long long num_tiles, long long total, int tile, int ddof, float eps,
                                 float* mean_rstd, cudaStream_t stream) {
    norm_finalize_kernel<<<1, 1024, 0, stream>>>(partial, num_tiles, total, tile, ddof, eps, mean_rstd);
    return cudaGetLastError();
}

cudaError_t launch_norm_rescale(float* adv, long long total, const float* mean_rstd, bool vec, cudaStream_t stream) {
    const long long blocks = (total + 2047) / 2048;
    if (vec) norm_rescale_kernel<true><<<(unsigned)blocks, 256, 0, stream>>>(adv, total, mean_rstd);
    else norm_rescale_kernel<false><<<(unsigned)blocks, 256, 0, stream>>>(adv, total, mean_rstd);
    return cudaGetLastError();
}

}  // namespace rlcs
