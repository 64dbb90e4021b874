// Vector-valued eligibility traces: x, z of shape [N, T, D] (d innermost), one scalar decay per
// step shared by all D components (Table 1, row "Elig. Traces", in its vector form), or -- PERDIM --
// a decay per component and step read from a [N, T, D] tensor (the per-dimension beta that true
// online TD(lambda) needs and Section 9.1 lists as unsupported by a scalar-beta kernel).
//
// The scan runs along T, which is the strided axis of this layout, so the mapping is the transpose of
// the flat-tile kernels: a thread owns 4 (or 1) adjacent components d of one row n and walks the
// timesteps in order -- z <- beta_t * z + x_t is one FMA per component -- while the 32 lanes of a
// warp cover adjacent components, so every load and store is a fully used 512-byte (or 128-byte)
// segment.  Addresses do not depend on the recurrence: UNROLL steps are loaded before the first
// FMA, which keeps UNROLL x 16 bytes per thread in flight.
//
// Parallelism is N * D/4 threads.  When that cannot fill the GPU (few long rows) the time axis is cut
// into chunks: pass 1 computes each chunk's end vector with carry 0 and its decay product, a small
// pass chains the carries of a row's chunks in order, and pass 3 rescans every chunk from its carry
// and writes the traces (x is then read twice).  Deterministic either way.
#include <cstdint>

#include "../../include/rlcs.h"
#include "rlcs_device.cuh"
#include "rlcs_scan.cuh"

// the time-major block kernel, one [T, D] problem per row (rlcs_time_major.cu)
namespace rlcs_internal {
bool vec_trace_block_usable(const float* x, const float* beta, int64_t N, int64_t T, int64_t D);
size_t vec_trace_block_workspace_bytes(int64_t N, int64_t T, int64_t D, bool perdim);
int vec_trace_block(const float* x, const float* beta, const uint8_t* dones, float* traces, int64_t N, int64_t T, int64_t D,
                    float decay, void* workspace, size_t workspace_bytes, void* cuda_stream);
}  // namespace rlcs_internal

namespace {

constexpr int kBatch = 8;         // steps loaded before the first FMA (x 16 bytes per thread in flight) ...
constexpr int kBatchMax = 32;     // ... up to this many when the threads are few
constexpr int kThreads = 256;
int g_force_batch = 0, g_force_chunks = 0;     // test hook: 0 = planned
bool g_force_block = false;                    // test hook: the time-major block kernel wherever usable

struct VecParams {
    const float* x;
    const uint8_t* dones;
    float* z;
    long long N;
    unsigned T, D;
    unsigned groups;          // threads per row: ceil(D / V)
    unsigned chunk;           // timesteps per chunk (== T when the time axis is not cut)
    unsigned batch;           // steps loaded before the first FMA: 8, 16 or 32 (per-component decay: half)
    unsigned chunks;          // chunks per row
    float decay;
    const float* beta;        // PERDIM: [N, T, D] decays; beta[n, t, :] multiplies z_{t-1} into step t
    float* ends;              // [N, chunks, D]: pass 1 chunk-end vectors, then (in place) the carries into each chunk
    float* prods;             // [N, chunks]: decay product of each chunk; PERDIM: [N, chunks, D]
};

template <int V> struct Vec;
template <> struct Vec<4> {
    float4 v;
    __device__ static Vec load(const float* p) { Vec r; r.v = __ldcs(reinterpret_cast<const float4*>(p)); return r; }
    __device__ static Vec plain(const float* p) { Vec r; r.v = *reinterpret_cast<const float4*>(p); return r; }
    __device__ void store(float* p) const { __stcs(reinterpret_cast<float4*>(p), v); }
    __device__ void plain_store(float* p) const { *reinterpret_cast<float4*>(p) = v; }
    __device__ static Vec zero() { Vec r; r.v = make_float4(0.f, 0.f, 0.f, 0.f); return r; }
    __device__ static Vec splat(float f) { Vec r; r.v = make_float4(f, f, f, f); return r; }
    __device__ void fma(float b, const Vec& x) {     // this <- b * this + x
        v.x = fmaf(b, v.x, x.v.x); v.y = fmaf(b, v.y, x.v.y); v.z = fmaf(b, v.z, x.v.z); v.w = fmaf(b, v.w, x.v.w);
    }
    __device__ void fma(const Vec& b, const Vec& x) {     // this <- b * this + x, component by component
        v.x = fmaf(b.v.x, v.x, x.v.x); v.y = fmaf(b.v.y, v.y, x.v.y); v.z = fmaf(b.v.z, v.z, x.v.z); v.w = fmaf(b.v.w, v.w, x.v.w);
    }
    __device__ void mul(const Vec& b) { v.x *= b.v.x; v.y *= b.v.y; v.z *= b.v.z; v.w *= b.v.w; }
    // zero unless on; bitwise, so that a flag that differs between the rows of a warp cannot become a branch
    __device__ void keep(bool on) {
        const unsigned m = on ? ~0u : 0u;
        v.x = __uint_as_float(__float_as_uint(v.x) & m); v.y = __uint_as_float(__float_as_uint(v.y) & m);
        v.z = __uint_as_float(__float_as_uint(v.z) & m); v.w = __uint_as_float(__float_as_uint(v.w) & m);
    }
};
template <> struct Vec<1> {
    float v;
    __device__ static Vec load(const float* p) { Vec r; r.v = __ldcs(p); return r; }
    __device__ static Vec plain(const float* p) { Vec r; r.v = *p; return r; }
    __device__ void store(float* p) const { __stcs(p, v); }
    __device__ void plain_store(float* p) const { *p = v; }
    __device__ static Vec zero() { Vec r; r.v = 0.f; return r; }
    __device__ static Vec splat(float f) { Vec r; r.v = f; return r; }
    __device__ void fma(float b, const Vec& x) { v = fmaf(b, v, x.v); }
    __device__ void fma(const Vec& b, const Vec& x) { v = fmaf(b.v, v, x.v); }
    __device__ void mul(const Vec& b) { v *= b.v; }
    __device__ void keep(bool on) { v = __uint_as_float(__float_as_uint(v) & (on ? ~0u : 0u)); }
};

// MODE 0: whole rows, write traces.  MODE 1: chunk ends and decay products only.  MODE 2: rescan
// from the carry and write traces.
template <int V, int MODE, bool PERDIM, int KB>
__global__ void __launch_bounds__(kThreads) elig_vec_kernel(const VecParams p) {
    const long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long per_row = (long long)p.groups * p.chunks;
    const long long n = tid / per_row;
    if (n >= p.N) return;
    const unsigned rest = (unsigned)(tid - n * per_row);
    const unsigned k = rest / p.groups;                       // chunk of the row
    const unsigned c = (rest - k * p.groups) * V;             // first component of this thread
    const unsigned t_begin = k * p.chunk;
    const unsigned t_end = min(p.T, t_begin + p.chunk);
    const long long row = n * (long long)p.T;
    const float* __restrict__ x = p.x + (row * p.D + c);
    float* __restrict__ z = p.z + (row * p.D + c);
    const uint8_t* __restrict__ d = p.dones + row;
    const float* __restrict__ bsrc = PERDIM ? p.beta + (row * p.D + c) : nullptr;

    Vec<V> acc = Vec<V>::zero();
    if (MODE == 2 && k > 0) acc = Vec<V>::plain(p.ends + ((n * p.chunks + k) * (long long)p.D + c));
    float prod = 1.f;                          // decay product of the chunk (scalar decay)
    Vec<V> prodv = Vec<V>::splat(1.f);         // ... per component (PERDIM)

    // (A software pipeline of two alternating register batches was measured and is slower: 0.60
    // against 0.89 of the copy bandwidth for the shared-decay kernel.)
    for (unsigned t0 = t_begin; t0 < t_end; t0 += KB) {
        Vec<V> xs[KB], bs[KB];
        float beta[KB];
#pragma unroll
        for (int u = 0; u < KB; ++u) {
            const unsigned t = t0 + u;
            if (t < t_end) {
                xs[u] = Vec<V>::load(x + (long long)t * p.D);
                // the carry into step t is severed by the flag of step t-1 (and at the row's first step)
                const bool cut = (t == 0 || __ldg(d + t - 1) != 0);
                if constexpr (PERDIM) {
                    bs[u] = Vec<V>::load(bsrc + (long long)t * p.D);
                    bs[u].keep(!cut);
                } else {
                    beta[u] = cut ? 0.f : p.decay;
                }
            }
        }
#pragma unroll
        for (int u = 0; u < KB; ++u) {
            const unsigned t = t0 + u;
            if (t < t_end) {
                if constexpr (PERDIM) {
                    acc.fma(bs[u], xs[u]);
                    if (MODE == 1) prodv.mul(bs[u]);
                } else {
                    acc.fma(beta[u], xs[u]);
                    if (MODE == 1) prod *= beta[u];
                }
                if (MODE != 1) acc.store(z + (long long)t * p.D);
            }
        }
    }
    if (MODE == 1) {
        acc.plain_store(p.ends + ((n * p.chunks + k) * (long long)p.D + c));
        if constexpr (PERDIM) prodv.plain_store(p.prods + ((n * p.chunks + k) * (long long)p.D + c));
        else if (c == 0) p.prods[n * p.chunks + k] = prod;
    }
}

// Chain the chunks of each row: carry into chunk k = end_{k-1} + prod_{k-1} * carry into chunk k-1,
// in order, one thread per (row, component group).  Overwrites ends[n][k] with the carry into chunk k.
template <int V, bool PERDIM>
__global__ void __launch_bounds__(kThreads) elig_vec_chain_kernel(const VecParams p) {
    const long long tid = (long long)blockIdx.x * kThreads + threadIdx.x;
    const long long n = tid / p.groups;
    if (n >= p.N) return;
    const unsigned c = (unsigned)(tid - n * p.groups) * V;
    float* e = p.ends + (n * p.chunks * (long long)p.D + c);
    const float* pr = PERDIM ? p.prods + (n * p.chunks * (long long)p.D + c) : p.prods + n * p.chunks;
    Vec<V> carry = Vec<V>::zero();
    for (unsigned k = 0; k < p.chunks; ++k) {
        const Vec<V> end_k = Vec<V>::plain(e + (long long)k * p.D);     // computed with carry 0
        carry.plain_store(e + (long long)k * p.D);                      // carry into chunk k
        if constexpr (PERDIM) carry.fma(Vec<V>::plain(pr + (long long)k * p.D), end_k);
        else carry.fma(pr[k], end_k);                                   // carry into chunk k+1
    }
}

inline bool aligned(const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

// How deep each thread loads ahead, and whether the time axis is cut.  One pass keeps
// threads x batch x 16 bytes in flight; about 300 K thread-steps (5 MB) saturate HBM with 8 steps per
// thread.  With fewer threads the batch grows to 32 steps (0.49 -> 0.81 of the copy bandwidth at
// 2048x512x64; 16 steps: 0.76); only when that is not enough is the time axis cut -- into chunks of
// at least 128 steps and at most 256 per row, so that the ordered carry chain stays short.
void plan(long long N, long long T, long long groups, bool perdim, unsigned* chunk, unsigned* chunks, unsigned* batch) {
    const long long want = rlcs_device::limits().sms * 256 * kBatch;
    const long long threads = N * groups;
    unsigned kb = kBatch;
    // (with a decay tensor the deeper batches measured slower: 0.87 -> 0.58 -> 0.38 at 16384x128x64)
    if (!perdim && threads * kb < want) kb = kBatchMax;
    if (g_force_batch) kb = (unsigned)g_force_batch;
    long long k = 1;
    if (threads * kb < want) { kb = g_force_batch ? kb : kBatch; k = (want + threads * kb - 1) / (threads * kb); }
    if (g_force_chunks) k = g_force_chunks;
    if (k > 256) k = 256;
    long long len = (T + k - 1) / k;
    if (len < 128) len = 128;
    len = (len + kBatchMax - 1) / kBatchMax * kBatchMax;
    *batch = kb;
    if (len >= T) { *chunk = (unsigned)T; *chunks = 1; return; }
    *chunk = (unsigned)len;
    *chunks = (unsigned)((T + len - 1) / len);
}

template <int V, bool PERDIM, int KB>
int run_batch(const VecParams& p, cudaStream_t s) {
    const long long threads = p.N * (long long)p.groups * p.chunks;
    // few threads: smaller blocks, so that they spread over all SMs
    const unsigned bt = threads < rlcs_device::limits().sms * kThreads * 2 ? 64 : kThreads;
    const unsigned blocks = (unsigned)((threads + bt - 1) / bt);
    if (p.chunks == 1) {
        elig_vec_kernel<V, 0, PERDIM, KB><<<blocks, bt, 0, s>>>(p);
    } else {
        elig_vec_kernel<V, 1, PERDIM, KB><<<blocks, bt, 0, s>>>(p);
        const long long chain_threads = p.N * (long long)p.groups;
        elig_vec_chain_kernel<V, PERDIM><<<(unsigned)((chain_threads + kThreads - 1) / kThreads), kThreads, 0, s>>>(p);
        elig_vec_kernel<V, 2, PERDIM, KB><<<blocks, bt, 0, s>>>(p);
    }
    return cudaGetLastError() == cudaSuccess ? RLCS_OK : RLCS_ERR_CUDA;
}

// the per-component decay loads two tensors per step: half the steps for the same bytes in flight
template <int V, bool PERDIM>
int run(const VecParams& p, cudaStream_t s) {
    constexpr int H = PERDIM ? 2 : 1;
    switch (p.batch) {
        case 32: return run_batch<V, PERDIM, 32 / H>(p, s);
        case 16: return run_batch<V, PERDIM, 16 / H>(p, s);
        default: return run_batch<V, PERDIM, 8 / H>(p, s);
    }
}

// sizes, pointers and chunking common to both entry points; *skip = nothing to do
int prepare(VecParams& p, const float* x, const float* beta, bool perdim, const uint8_t* dones, float* traces, int64_t N,
            int64_t T, int64_t D, void* workspace, size_t workspace_bytes, bool* v4, bool* skip) {
    *skip = false;
    if (N < 0 || T < 0 || D < 0 || T > (int64_t(1) << 31) - 1 || D > (int64_t(1) << 24)) return RLCS_ERR_SIZE;
    if (N == 0 || T == 0 || D == 0) { *skip = true; return RLCS_OK; }
    if (N > (int64_t(1) << 40) / T || N * T > (int64_t(1) << 40) / D) return RLCS_ERR_SIZE;
    if (!x || !dones || !traces || (perdim && !beta)) return RLCS_ERR_NULL;
    if (!aligned(x, 4) || !aligned(traces, 4) || (perdim && !aligned(beta, 4))) return RLCS_ERR_ALIGN;
    *v4 = (D % 4 == 0) && aligned(x, 16) && aligned(traces, 16) && (!perdim || aligned(beta, 16));
    p.x = x; p.beta = beta; p.dones = dones; p.z = traces; p.N = N; p.T = (unsigned)T; p.D = (unsigned)D;
    p.groups = (unsigned)(*v4 ? D / 4 : D);
    plan(N, T, p.groups, perdim, &p.chunk, &p.chunks, &p.batch);
    if (p.chunks > 1) {
        const size_t need = sizeof(float) * (size_t)N * p.chunks * ((size_t)D + (perdim ? (size_t)D : 1));
        if (workspace == nullptr || workspace_bytes < need) return RLCS_ERR_WORKSPACE;
        if (!aligned(workspace, 16)) return RLCS_ERR_ALIGN;
        p.ends = static_cast<float*>(workspace);
        p.prods = p.ends + (size_t)N * p.chunks * (size_t)D;
    }
    return RLCS_OK;
}

size_t workspace_bytes(int64_t N, int64_t T, int64_t D, bool perdim) {
    if (N <= 0 || T <= 0 || D <= 0 || T > (int64_t(1) << 31) - 1 || D > (int64_t(1) << 24)) return 0;
    unsigned chunk, chunks, batch;
    plan(N, T, (D + 3) / 4, perdim, &chunk, &chunks, &batch);
    unsigned chunk1, chunks1;
    plan(N, T, D, perdim, &chunk1, &chunks1, &batch);                         // the element-wise variant cuts differently
    const size_t k = chunks > chunks1 ? chunks : chunks1;
    const size_t walk = k <= 1 ? 0 : sizeof(float) * (size_t)N * k * ((size_t)D + (perdim ? (size_t)D : 1)) + 256;
    const size_t block = rlcs_internal::vec_trace_block_workspace_bytes(N, T, D, perdim);   // the block kernel's chained chunks
    return walk > block ? walk : block;
}

}  // namespace

extern "C" {

size_t rlcs_elig_trace_vec_workspace_bytes(int64_t N, int64_t T, int64_t D) { return workspace_bytes(N, T, D, false); }

size_t rlcs_elig_trace_vec_beta_workspace_bytes(int64_t N, int64_t T, int64_t D) { return workspace_bytes(N, T, D, true); }

int rlcs_elig_trace_vec(const float* x, const uint8_t* dones, float* traces, int64_t N, int64_t T, int64_t D,
                        float gamma, float lambda, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (!(gamma >= 0.f && gamma <= 1.f) || !(lambda >= 0.f && lambda <= 1.f)) return RLCS_ERR_ARG;
    VecParams p = {};
    bool v4 = false, skip = false;
    const int st = prepare(p, x, nullptr, false, dones, traces, N, T, D, workspace, workspace_bytes, &v4, &skip);
    if (st != RLCS_OK || skip) return st;
    p.decay = gamma * lambda;
    // Below the sizes that fill the GPU with one thread per four components the time-major block kernel
    // (one block per row and 32 components, x read from HBM once) is faster: 0.56 -> 0.63 of the copy
    // bandwidth at 1024x1024x64, 0.44 -> 0.62 at 512x2048x64; for few long rows it cuts the time axis
    // and chains the chunks in one launch (0.41 -> 0.46 at 64x16384x64, against the three-launch
    // chunked walk below, which reads x twice and remains for shapes the block kernel cannot take).
    const bool mid = (long long)N * p.groups < 32768;
    if ((mid || g_force_block) && !g_force_batch && !g_force_chunks && rlcs_internal::vec_trace_block_usable(x, nullptr, N, T, D))
        return rlcs_internal::vec_trace_block(x, nullptr, dones, traces, N, T, D, p.decay, workspace, workspace_bytes, cuda_stream);
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    return v4 ? run<4, false>(p, s) : run<1, false>(p, s);
}

int rlcs_elig_trace_vec_beta(const float* x, const float* beta, const uint8_t* dones, float* traces, int64_t N, int64_t T,
                             int64_t D, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    VecParams p = {};
    bool v4 = false, skip = false;
    const int st = prepare(p, x, beta, true, dones, traces, N, T, D, workspace, workspace_bytes, &v4, &skip);
    if (st != RLCS_OK || skip) return st;
    // Wherever its copies can be issued (D a multiple of 4 and >= 32, 16-byte aligned tensors) the
    // time-major block kernel streams each row once and is at least as fast as the thread-per-four-
    // components walk: 0.87 -> 0.92 of the copy bandwidth at 16384x128x64, 0.63 -> 0.90 at 4096x512x64,
    // 0.21 -> 0.47 at 64x16384x64 (where the walk would have to cut the time axis and read twice).
    if (!g_force_batch && !g_force_chunks && rlcs_internal::vec_trace_block_usable(x, beta, N, T, D))
        return rlcs_internal::vec_trace_block(x, beta, dones, traces, N, T, D, 1.f, workspace, workspace_bytes, cuda_stream);
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    return v4 ? run<4, true>(p, s) : run<1, true>(p, s);
}

void rlcs_debug_vec_trace_plan(int batch, int chunks) {
    g_force_batch = (batch == 8 || batch == 16 || batch == 32) ? batch : 0;
    g_force_block = batch == 1;
    g_force_chunks = chunks > 0 ? chunks : 0;
}

}  // extern "C"
