// GAE with advantage normalisation: the GAE scan kernel that also leaves per-tile sums, a one-block
// reduction of those sums to mean and 1/(std + eps), and the element-wise rescale of the advantages.
#include "rlcs_launch.cuh"

namespace rlcs {

RLCS_DEFINE_LAUNCHER(launch_gae_stats, kGaeStats, true)

// One block: per-tile partial sums -> {mean, 1/(std + eps)}.  Each thread adds its strided share in
// double, then a shared-memory tree in a fixed order: the result does not depend on timing.
__global__ void __launch_bounds__(1024) norm_finalize_kernel(const float* __restrict__ partial, long long num_tiles,
                                                             double count, int ddof, float eps, float* __restrict__ out) {
    __shared__ double sh1[1024], sh2[1024];
    double s1 = 0.0, s2 = 0.0;
    for (long long i = threadIdx.x; i < num_tiles; i += 1024) {
        s1 += (double)partial[2 * i];
        s2 += (double)partial[2 * i + 1];
    }
    sh1[threadIdx.x] = s1;
    sh2[threadIdx.x] = s2;
    __syncthreads();
    for (int d = 512; d > 0; d >>= 1) {
        if ((int)threadIdx.x < d) {
            sh1[threadIdx.x] += sh1[threadIdx.x + d];
            sh2[threadIdx.x] += sh2[threadIdx.x + d];
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        const double mean = sh1[0] / count;
        const double denom = count - (double)ddof;
        double var = denom > 0.0 ? (sh2[0] - sh1[0] * mean) / denom : 0.0;     // sum (A - mean)^2 = sum A^2 - mean * sum A
        if (var < 0.0) var = 0.0;
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

cudaError_t launch_norm_finalize(const float* partial, long long num_tiles, double count, int ddof, float eps,
                                 float* mean_rstd, cudaStream_t stream) {
    norm_finalize_kernel<<<1, 1024, 0, stream>>>(partial, num_tiles, count, ddof, eps, mean_rstd);
    return cudaGetLastError();
}

cudaError_t launch_norm_rescale(float* adv, long long total, const float* mean_rstd, bool vec, cudaStream_t stream) {
    const long long blocks = (total + 2047) / 2048;
    if (vec) norm_rescale_kernel<true><<<(unsigned)blocks, 256, 0, stream>>>(adv, total, mean_rstd);
    else norm_rescale_kernel<false><<<(unsigned)blocks, 256, 0, stream>>>(adv, total, mean_rstd);
    return cudaGetLastError();
}

}  // namespace rlcs
