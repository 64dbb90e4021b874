// Fused segmented affine scan over the flattened [N*T] rollout array (sm_100a).
//
// One kernel template serves all seven algorithms.  The row-major [N, T] tensors are treated as
// one contiguous array of N*T steps that is cut into fixed tiles of THREADS*ITEMS steps, one
// thread block per tile; a row edge is simply one more reset.  Per tile:
//   1. every thread loads ITEMS consecutive steps of each input with 16-byte vector loads
//      (masks: one ITEMS-byte load), plus a one-step halo of the successor value;
//   2. builds (alpha_t, beta_t) of Table 1 in registers, with the boundary rules of Section 3.2
//      and the window-edge carry folded into alpha, so that every row scans with carry 0;
//   3. folds its ITEMS pairs serially with the combine of Eq. 2, scans the per-thread aggregates
//      with warp shuffles, and the per-warp aggregates through shared memory;
//   4. if the tile is entered in the middle of an episode, obtains the carry from the preceding
//      tiles (in scan order) by a bounded, deterministic look-back over published tile aggregates;
//   5. replays the recurrence over its ITEMS steps from the carry, applies the epilogue
//      (returns = A + V, V-Trace targets and advantages, Retrace targets) and stores once.
// Backward algorithms scan from high addresses to low ones; thread block s handles tile
// num_tiles-1-s, so that a block only ever waits on blocks with a smaller block index.
//
// The kernel is bound by HBM traffic and, next, by integer/select issue slots, so the per-step
// code is branch-free: flags stay packed as mask bytes (4 steps per 32-bit word), a reset is a
// beta of exactly 0 (0 * finite = 0 severs exactly), and the rare cases -- a row edge inside a
// thread's chunk, the ragged last chunk, rows shorter than a chunk -- patch the packed words in
// short side paths.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace rlcs {

enum Algo : int {
    kGae = 0, kTdLambda = 1, kDisc = 2, kVtrace = 3, kRetrace = 4, kElig = 5, kPrefix = 6,
    kAffineBwd = 7, kAffineFwd = 8
};

__host__ __device__ constexpr bool is_forward(int a) { return a == kElig || a == kPrefix || a == kAffineFwd; }
__host__ __device__ constexpr bool has_values(int a) { return a == kGae || a == kTdLambda || a == kVtrace; }
__host__ __device__ constexpr bool is_affine(int a) { return a == kAffineBwd || a == kAffineFwd; }
__host__ __device__ constexpr bool const_decay(int a) { return a != kVtrace && a != kRetrace && !is_affine(a); }

constexpr unsigned kDeviceTimeout = 7;   // RLCS_ERR_TIMEOUT
constexpr int kHeaderWords = 64;         // workspace header: 256 bytes
// header[0] = call counter (epoch), header[1] = finished-block counter, header[2] = status word

// Division of a 32-bit index by the invariant row length T (Granlund-Montgomery, round-up form):
// q = (hi + ((n - hi) >> sh1)) >> sh2 with hi = umulhi(mul, n).  Exact for every n < 2^32, T >= 1.
struct FastDiv {
    unsigned mul, sh1, sh2;
};

struct ScanParams {
    const float* f0;          // rewards | x | alpha
    const float* f1;          // values | q_sa | beta
    const float* f2;          // expected_q
    const float* f3;          // log_rhos
    const uint8_t* dones;
    const uint8_t* truncs;
    const float* trunc_boot;  // [N,T]
    const float* boot;        // [N] or nullptr
    float* out0;
    float* out1;              // second output or nullptr
    long long total;          // N*T
    long long num_tiles;
    unsigned T;
    int idx32;                // total + tile fits in 32 bits: 32-bit row/time arithmetic
    FastDiv div_T;
    float gamma;
    float decay;              // gamma*lambda | gamma | 1
    float decay_pow;          // decay^ITEMS: the beta product of a chunk without resets
    float aux;                // TD(lambda): gamma*(1-lambda); Retrace: gamma*lambda
    float rho_bar, c_bar;
    int starts_at;
    int carry_mode;           // rows may straddle tiles: publish aggregates, look back
    unsigned* header;
    uint4* records;           // one 16-byte record per tile: {alpha_bits, epoch, beta_bits, epoch}
    long long mute_tile;      // test hook: this scan-order tile does not publish
    unsigned spin_cap;
};

struct Pair { float a, b; };

// `x` covers steps that come later in scan order than everything in `acc`:
// result = x (+) acc = (x.a + x.b*acc.a, x.b*acc.b)  (Eq. 2).
__device__ __forceinline__ Pair apply(Pair x, Pair acc) {
    Pair r;
    r.a = fmaf(x.b, acc.a, x.a);
    r.b = x.b * acc.b;
    return r;
}

// ------------------------------------------------------------------------------------------ loads / stores
template <int ITEMS, bool VEC>
__device__ __forceinline__ void load_f32(const float* __restrict__ p, long long i0, int nvalid, float (&x)[ITEMS]) {
    if (VEC && nvalid == ITEMS) {
        const float4* q = reinterpret_cast<const float4*>(p + i0);
#pragma unroll
        for (int k = 0; k < ITEMS / 4; ++k) {
            float4 v = __ldcs(q + k);
            x[4 * k + 0] = v.x; x[4 * k + 1] = v.y; x[4 * k + 2] = v.z; x[4 * k + 3] = v.w;
        }
    } else {
#pragma unroll
        for (int j = 0; j < ITEMS; ++j) x[j] = (j < nvalid) ? __ldcs(p + i0 + j) : 0.f;
    }
}

// Mask bytes of ITEMS consecutive steps, packed 4 per word (byte j%4 of word j/4), values as stored
// (any non-zero byte = true).
template <int ITEMS, bool VEC>
__device__ __forceinline__ void load_mask(const uint8_t* __restrict__ p, long long i0, int nvalid, unsigned (&w)[ITEMS / 4]) {
    if (VEC && nvalid == ITEMS) {
        if constexpr (ITEMS == 4) {
            w[0] = __ldcs(reinterpret_cast<const unsigned*>(p + i0));
        } else if constexpr (ITEMS == 8) {
            uint2 v = __ldcs(reinterpret_cast<const uint2*>(p + i0));
            w[0] = v.x; w[1] = v.y;
        } else {
            static_assert(ITEMS == 16, "ITEMS must be 4, 8 or 16");
            uint4 v = __ldcs(reinterpret_cast<const uint4*>(p + i0));
            w[0] = v.x; w[1] = v.y; w[2] = v.z; w[3] = v.w;
        }
    } else {
#pragma unroll
        for (int k = 0; k < ITEMS / 4; ++k) w[k] = 0;
#pragma unroll
        for (int j = 0; j < ITEMS; ++j)
            if (j < nvalid) w[j / 4] |= (unsigned)__ldcs(p + i0 + j) << (8 * (j % 4));
    }
}

template <int ITEMS, bool VEC>
__device__ __forceinline__ void store_f32(float* __restrict__ p, long long i0, int nvalid, const float (&x)[ITEMS]) {
    if (VEC && nvalid == ITEMS) {
        float4* q = reinterpret_cast<float4*>(p + i0);
#pragma unroll
        for (int k = 0; k < ITEMS / 4; ++k)
            __stcs(q + k, make_float4(x[4 * k + 0], x[4 * k + 1], x[4 * k + 2], x[4 * k + 3]));
    } else {
#pragma unroll
        for (int j = 0; j < ITEMS; ++j)
            if (j < nvalid) __stcs(p + i0 + j, x[j]);
    }
}

// ------------------------------------------------------------------------------------------ packed mask bytes
__device__ __forceinline__ constexpr unsigned byte_mask(int j) { return 0xffu << (8 * (j % 4)); }

template <int W>
__device__ __forceinline__ bool test_byte(const unsigned (&w)[W], int j) {      // j is a compile-time constant after unrolling
    return (w[j / 4] & byte_mask(j)) != 0;
}
template <int W>
__device__ __forceinline__ void mark_byte_dyn(unsigned (&w)[W], unsigned j) {   // j known only at run time
#pragma unroll
    for (int k = 0; k < W; ++k) w[k] |= ((j >> 2) == (unsigned)k) ? (0xffu << ((j & 3u) * 8u)) : 0u;
}
template <int W>
__device__ __forceinline__ bool test_byte_dyn(const unsigned (&w)[W], unsigned j) {
    unsigned v = 0;
#pragma unroll
    for (int k = 0; k < W; ++k) v |= ((j >> 2) == (unsigned)k) ? w[k] : 0u;
    return ((v >> ((j & 3u) * 8u)) & 0xffu) != 0;
}

// ------------------------------------------------------------------------------------------ tile records
__device__ __forceinline__ uint4 ld_volatile_u4(const uint4* p) {
    uint4 v;
    asm volatile("ld.volatile.global.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_volatile_u4(uint4* p, uint4 v) {
    asm volatile("st.volatile.global.v4.u32 [%0], {%1,%2,%3,%4};"
                 :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ unsigned ld_volatile_u32(const unsigned* p) {
    unsigned v;
    asm volatile("ld.volatile.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Carry into scan-order tile `s`: the recurrence value at the last step (in scan order) of tile
// s-1, i.e. the fold  a_{s-1} + b_{s-1}*(a_{s-2} + b_{s-2}*(...))  of the published tile
// aggregates, cut at the first aggregate whose beta is zero (a reset, or the row edge, inside that
// tile).  Only aggregates are folded, always in this fixed order, so the result does not depend on
// timing.  One warp runs this; each lane polls one predecessor.  Each 16-byte record carries the
// call's epoch next to each 4-byte payload word, so an 8-byte half is self-validating and no
// fence is needed.  The wait is bounded: after `cap` polls the status word is set and 0 returned.
static __device__ __noinline__ float lookback(const uint4* __restrict__ records, unsigned epoch, long long s,
                                       unsigned cap, unsigned* status, int lane) {
    Pair acc = {0.f, 1.f};
    long long base = s - 1;
    unsigned polls = 0;
    for (;;) {
        const long long idx = base - lane;
        Pair p = {0.f, 0.f};          // a tile before the first one: a terminator
        bool ready = true;
        if (idx >= 0) {
            uint4 v = ld_volatile_u4(records + idx);
            ready = (v.y == epoch) && (v.w == epoch);
            p.a = __uint_as_float(v.x);
            p.b = __uint_as_float(v.z);
        }
        const unsigned rdy = __ballot_sync(0xffffffffu, ready);
        const unsigned zer = __ballot_sync(0xffffffffu, ready && p.b == 0.f);
        const int n_ready = (rdy == 0xffffffffu) ? 32 : (__ffs(~rdy) - 1);   // ready lanes 0..n_ready-1
        const int z = zer ? (__ffs(zer) - 1) : 32;                           // first terminator
        const bool done = z < n_ready;
        if (!done && n_ready < 32) {
            if (++polls > cap) {
                if (lane == 0) atomicExch(status, kDeviceTimeout);
                return 0.f;
            }
            __nanosleep(32);
            continue;
        }
        // fold lanes 0..min(z,31) in lane order (lane 0 = nearest tile); a terminator's alpha is
        // taken as is, nothing beyond it is touched
        Pair cur = (lane <= z) ? p : Pair{0.f, 1.f};
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            Pair o;
            o.a = __shfl_down_sync(0xffffffffu, cur.a, d);
            o.b = __shfl_down_sync(0xffffffffu, cur.b, d);
            if (lane + d < 32 && cur.b != 0.f) cur = apply(cur, o);
        }
        Pair w;
        w.a = __shfl_sync(0xffffffffu, cur.a, 0);
        w.b = __shfl_sync(0xffffffffu, cur.b, 0);
        acc = apply(acc, w);
        if (done) return acc.a;
        base -= 32;
    }
}

// ------------------------------------------------------------------------------------------ the kernel
template <int ALGO, bool TRUNC, bool VEC, int THREADS, int ITEMS, int MIN_BLOCKS>
__global__ void __launch_bounds__(THREADS, MIN_BLOCKS) scan_kernel(const ScanParams p) {
    constexpr bool FWD = is_forward(ALGO);
    constexpr int NW = THREADS / 32;
    constexpr int W = ITEMS / 4;
    constexpr int TILE = THREADS * ITEMS;
    constexpr unsigned FULL = 0xffffffffu;
    static_assert(NW <= 32 && ITEMS % 4 == 0, "bad tile shape");

    __shared__ Pair s_agg[NW];     // warp aggregates, indexed by the warp's rank in scan order
    __shared__ float s_carry;      // tile carry-in
    __shared__ int s_need;         // the tile is entered mid-episode

    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int warp = tid >> 5;
    const long long s = blockIdx.x;                       // tile index in scan order
    const long long tile = FWD ? s : (p.num_tiles - 1 - s);
    const long long i0 = tile * TILE + (long long)tid * ITEMS;
    const long long rem = p.total - i0;
    const int nvalid = rem >= ITEMS ? ITEMS : (rem > 0 ? (int)rem : 0);

    // row and timestep of this thread's first step
    long long n0;
    unsigned t0;
    if (p.idx32) {
        const unsigned n = (unsigned)i0;
        const unsigned hi = __umulhi(p.div_T.mul, n);
        const unsigned q = (hi + ((n - hi) >> p.div_T.sh1)) >> p.div_T.sh2;
        n0 = q;
        t0 = n - q * p.T;
    } else {
        n0 = i0 / (long long)p.T;
        t0 = (unsigned)(i0 - n0 * (long long)p.T);
    }

    // ------------------------------------------------------------------ 1. loads (all issued up front)
    unsigned dw[W], tw[W];
#pragma unroll
    for (int k = 0; k < W; ++k) { dw[k] = 0; tw[k] = 0; }
    if constexpr (!is_affine(ALGO)) load_mask<ITEMS, VEC>(p.dones, i0, nvalid, dw);
    if constexpr (TRUNC) load_mask<ITEMS, VEC>(p.truncs, i0, nvalid, tw);

    float alpha[ITEMS];            // rewards | x | alpha, then alpha_t, then the first output
    load_f32<ITEMS, VEC>(p.f0, i0, nvalid, alpha);
    float x1[ITEMS];               // values | q_sa | beta
    if constexpr (ALGO != kDisc && ALGO != kElig && ALGO != kPrefix) load_f32<ITEMS, VEC>(p.f1, i0, nvalid, x1);
    float x2[ITEMS];               // expected_q
    if constexpr (ALGO == kRetrace) load_f32<ITEMS, VEC>(p.f2, i0, nvalid, x2);
    float x3[ITEMS];               // log_rhos
    if constexpr (ALGO == kVtrace || ALGO == kRetrace) load_f32<ITEMS, VEC>(p.f3, i0, nvalid, x3);

    // one-step halo beyond the thread's chunk, in the direction of the dependency
    float halo = 0.f, halo_lr = 0.f;
    unsigned halo_d = 0;
    if constexpr (!FWD && (has_values(ALGO) || ALGO == kRetrace)) {
        const float* src = (ALGO == kRetrace) ? p.f2 : p.f1;
        const bool edge_lane = (lane == 31) && (rem > ITEMS);
        if (edge_lane) halo = __ldg(src + i0 + ITEMS);
        if constexpr (ALGO == kRetrace) if (edge_lane) halo_lr = __ldg(p.f3 + i0 + ITEMS);
    }
    if constexpr (ALGO == kElig || ALGO == kPrefix) {
        if (lane == 0 && i0 > 0 && rem > 0) halo_d = __ldg(p.dones + i0 - 1);
    }

    // Row edge inside the chunk.  Backward: the row's last step, at chunk offset T-1-t0; its
    // window-edge bootstrap is fetched now.  Forward: the next row's first step, at offset T-t0
    // (offset 0 when the chunk itself starts a row).
    const unsigned edge = FWD ? (t0 == 0 ? 0u : p.T - t0) : (p.T - 1 - t0);
    const bool has_edge = edge < (unsigned)ITEMS;
    float boot_first = 0.f;
    if constexpr (!FWD && !is_affine(ALGO)) {
        if (p.boot != nullptr && edge < (unsigned)nvalid) boot_first = __ldg(p.boot + n0);
    }

    // ------------------------------------------------------------------ 2. reset words
    // sev: byte j non-zero = the recurrence does NOT continue from step j to its scan-order
    // predecessor (t+1 backward, t-1 forward): a flag, a row edge, or a step beyond the array.
    unsigned sev[W];
    if constexpr (FWD) {
        if constexpr (ALGO == kAffineFwd) {
#pragma unroll
            for (int k = 0; k < W; ++k) sev[k] = 0;
        } else {
            // ends_at: step j is cut off by the flag of step j-1 -> shift the bytes up by one step
            const unsigned nb = __shfl_up_sync(FULL, dw[W - 1] >> 24, 1);
            if (lane != 0) halo_d = nb;
            if (ALGO == kPrefix && p.starts_at) {
#pragma unroll
                for (int k = 0; k < W; ++k) sev[k] = dw[k];
            } else {
#pragma unroll
                for (int k = 0; k < W; ++k) sev[k] = (dw[k] << 8) | (k == 0 ? (halo_d & 0xffu) : (dw[(k + W - 1) % W] >> 24));
            }
        }
    } else {
#pragma unroll
        for (int k = 0; k < W; ++k) sev[k] = dw[k] | tw[k];
    }
    if (has_edge) mark_byte_dyn(sev, edge);
    if (p.T < (unsigned)ITEMS) {                // rows shorter than a chunk: several edges
        for (unsigned e = edge + p.T; e < (unsigned)ITEMS; e += p.T) mark_byte_dyn(sev, e);
    }
    if (nvalid < ITEMS) {                       // ragged end of the array
        for (unsigned j = nvalid; j < (unsigned)ITEMS; ++j) mark_byte_dyn(sev, j);
    }

    // ------------------------------------------------------------------ 3. successor values at resets
    // ov[j]: successor value used where the recurrence is severed -- 0 after a termination, the
    // supplied continuation value after a truncation, the window-edge bootstrap at a row's last
    // step (Section 3.2).  Zero wherever the recurrence continues.
    float ov[ITEMS];
#pragma unroll
    for (int j = 0; j < ITEMS; ++j) ov[j] = 0.f;
    if constexpr (!FWD && !is_affine(ALGO)) {
        if constexpr (TRUNC) {
#pragma unroll
            for (int j = 0; j < ITEMS; ++j)
                if (test_byte(tw, j) && !test_byte(dw, j)) ov[j] = __ldg(p.trunc_boot + i0 + j);
        }
        if (has_edge && p.boot != nullptr) {
            unsigned e = edge;
            long long n = n0;
            float b = boot_first;
            for (;;) {
                if (e < (unsigned)nvalid && !test_byte_dyn(dw, e) && !test_byte_dyn(tw, e)) {
#pragma unroll
                    for (int j = 0; j < ITEMS; ++j) if ((unsigned)j == e) ov[j] = b;
                }
                e += p.T;
                ++n;
                if (e >= (unsigned)nvalid) break;          // only when T < ITEMS
                b = __ldg(p.boot + n);
            }
        }
    }

    // neighbour values through the warp
    if constexpr (!FWD && (has_values(ALGO) || ALGO == kRetrace)) {
        const float first = (ALGO == kRetrace) ? x2[0] : x1[0];
        const float nb = __shfl_down_sync(FULL, first, 1);
        if (lane != 31) halo = nb;
        if constexpr (ALGO == kRetrace) {
            const float nl = __shfl_down_sync(FULL, x3[0], 1);
            if (lane != 31) halo_lr = nl;
        }
    }

    // ------------------------------------------------------------------ 4. coefficients (branch-free)
    float beta[ITEMS];
    float grho[ITEMS];             // V-Trace: cont * gamma * rho_t, for the advantage epilogue
#pragma unroll
    for (int j = 0; j < ITEMS; ++j) {
        const bool cut = test_byte(sev, j);
        if constexpr (FWD) {
            if constexpr (ALGO == kAffineFwd) beta[j] = cut ? 0.f : x1[j];
            else beta[j] = cut ? 0.f : p.decay;
        } else if constexpr (ALGO == kAffineBwd) {
            beta[j] = cut ? 0.f : x1[j];
        } else {
            const float c = cut ? 0.f : 1.f;
            const float r = alpha[j];
            float nextv = 0.f;
            if constexpr (has_values(ALGO)) nextv = (j + 1 < ITEMS) ? x1[(j + 1) % ITEMS] : halo;
            if constexpr (ALGO == kRetrace) nextv = (j + 1 < ITEMS) ? x2[(j + 1) % ITEMS] : halo;
            if constexpr (ALGO == kGae) {
                alpha[j] = fmaf(p.gamma, fmaf(c, nextv, ov[j]), r) - x1[j];
                beta[j] = cut ? 0.f : p.decay;
            } else if constexpr (ALGO == kTdLambda) {
                // continuing: r + gamma(1-lambda) V_{t+1}; severed: r + gamma * successor value
                alpha[j] = fmaf(p.gamma, ov[j], fmaf(cut ? 0.f : p.aux, nextv, r));
                beta[j] = cut ? 0.f : p.decay;
            } else if constexpr (ALGO == kDisc) {
                alpha[j] = fmaf(p.gamma, ov[j], r);
                beta[j] = cut ? 0.f : p.decay;
            } else if constexpr (ALGO == kVtrace) {
                const float raw = expf(x3[j]);
                const float rho = fminf(p.rho_bar, raw);
                const float cc = fminf(p.c_bar, raw);
                alpha[j] = rho * (fmaf(p.gamma, fmaf(c, nextv, ov[j]), r) - x1[j]);
                beta[j] = cut ? 0.f : p.gamma * cc;
                grho[j] = cut ? 0.f : p.gamma * rho;
            } else if constexpr (ALGO == kRetrace) {
                alpha[j] = fmaf(p.gamma, fmaf(c, nextv, ov[j]), r) - x1[j];
                const float lr_next = (j + 1 < ITEMS) ? x3[(j + 1) % ITEMS] : halo_lr;
                beta[j] = cut ? 0.f : p.aux * fminf(p.c_bar, expf(lr_next));
            }
        }
    }

    // ------------------------------------------------------------------ 5. thread aggregate (serial combine, Eq. 2)
    Pair agg;
    if constexpr (FWD) {
        agg.a = alpha[0];
#pragma unroll
        for (int j = 1; j < ITEMS; ++j) agg.a = fmaf(beta[j], agg.a, alpha[j]);
    } else {
        agg.a = alpha[ITEMS - 1];
#pragma unroll
        for (int j = ITEMS - 2; j >= 0; --j) agg.a = fmaf(beta[j], agg.a, alpha[j]);
    }
    if constexpr (const_decay(ALGO)) {
        unsigned any = 0;
#pragma unroll
        for (int k = 0; k < W; ++k) any |= sev[k];
        agg.b = any ? 0.f : p.decay_pow;
    } else {
        agg.b = beta[0];
#pragma unroll
        for (int j = 1; j < ITEMS; ++j) agg.b *= beta[j];
    }

    // ------------------------------------------------------------------ 6. warp scan in scan order
    // rank = position in scan order inside the warp: lane for forward scans, 31 - lane for backward.
    const int rank = FWD ? lane : 31 - lane;
    Pair incl = agg;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        Pair o;
        if constexpr (FWD) {
            o.a = __shfl_up_sync(FULL, incl.a, d);
            o.b = __shfl_up_sync(FULL, incl.b, d);
        } else {
            o.a = __shfl_down_sync(FULL, incl.a, d);
            o.b = __shfl_down_sync(FULL, incl.b, d);
        }
        if (rank >= d) incl = apply(incl, o);
    }
    Pair excl;     // everything earlier in scan order inside this warp
    if constexpr (FWD) {
        excl.a = __shfl_up_sync(FULL, incl.a, 1);
        excl.b = __shfl_up_sync(FULL, incl.b, 1);
    } else {
        excl.a = __shfl_down_sync(FULL, incl.a, 1);
        excl.b = __shfl_down_sync(FULL, incl.b, 1);
    }
    if (rank == 0) excl = Pair{0.f, 1.f};

    // ------------------------------------------------------------------ 7. block carry through shared memory
    const int wrank = FWD ? warp : NW - 1 - warp;
    if (rank == 31) s_agg[wrank] = incl;
    if (wrank == 0 && rank == 0) {
        // the tile's first step in scan order: does the recurrence enter the tile from outside?
        s_need = test_byte(sev, FWD ? 0 : ITEMS - 1) ? 0 : 1;
    }
    __syncthreads();

    Pair wcarry = {0.f, 1.f};      // all warps earlier in scan order
    Pair tile_agg;
    {
        Pair w = (lane < NW) ? s_agg[lane] : Pair{0.f, 1.f};
#pragma unroll
        for (int d = 1; d < NW; d <<= 1) {
            Pair o;
            o.a = __shfl_up_sync(FULL, w.a, d);
            o.b = __shfl_up_sync(FULL, w.b, d);
            if (lane >= d) w = apply(w, o);
        }
        tile_agg.a = __shfl_sync(FULL, w.a, NW - 1);
        tile_agg.b = __shfl_sync(FULL, w.b, NW - 1);
        const float ca = __shfl_sync(FULL, w.a, (wrank + NW - 1) % NW);
        const float cb = __shfl_sync(FULL, w.b, (wrank + NW - 1) % NW);
        if (wrank > 0) wcarry = Pair{ca, cb};
    }
    const Pair before = apply(excl, wcarry);   // everything earlier in scan order inside this tile

    // ------------------------------------------------------------------ 8. carry between thread blocks
    float carry_in = 0.f;
    if (p.carry_mode) {
        unsigned epoch = 0;
        if (warp == 0) {
            epoch = ld_volatile_u32(p.header);
            if (lane == 0 && s != p.mute_tile) {
                st_volatile_u4(p.records + s, make_uint4(__float_as_uint(tile_agg.a), epoch,
                                                         __float_as_uint(tile_agg.b), epoch));
            }
        }
        const int need = s_need;               // block-uniform
        if (need) {
            if (warp == 0) {
                const float c = lookback(p.records, epoch, s, p.spin_cap, p.header + 2, lane);
                if (lane == 0) s_carry = c;
            }
            __syncthreads();
            carry_in = s_carry;
        }
    }
    // value of the recurrence at the step just before this thread's chunk in scan order
    float prev = fmaf(before.b, carry_in, before.a);

    // ------------------------------------------------------------------ 9. replay, epilogue, store
    float out1v[ITEMS];
    if constexpr (FWD) {
#pragma unroll
        for (int j = 0; j < ITEMS; ++j) {
            prev = fmaf(beta[j], prev, alpha[j]);
            alpha[j] = prev;
        }
    } else {
#pragma unroll
        for (int j = ITEMS - 1; j >= 0; --j) {
            const float d = fmaf(beta[j], prev, alpha[j]);
            if constexpr (ALGO == kGae) {
                alpha[j] = d;
                out1v[j] = d + x1[j];
            } else if constexpr (ALGO == kVtrace) {
                // A_t = rho_t (r_t + gamma v_{t+1} - V_t) = alpha_t + gamma rho_t Delta_{t+1} where the
                // recurrence continues (v_{t+1} = V_{t+1} + Delta_{t+1}), alpha_t elsewhere.
                out1v[j] = fmaf(grho[j], prev, alpha[j]);
                alpha[j] = x1[j] + d;
            } else if constexpr (ALGO == kRetrace) {
                alpha[j] = x1[j] + d;
            } else {
                alpha[j] = d;
            }
            prev = d;
        }
    }
    if (nvalid > 0) {
        store_f32<ITEMS, VEC>(p.out0, i0, nvalid, alpha);
        if constexpr (ALGO == kGae || ALGO == kVtrace) {
            if (p.out1 != nullptr) store_f32<ITEMS, VEC>(p.out1, i0, nvalid, out1v);
        }
    }

    // ------------------------------------------------------------------ 10. close the call (carry mode)
    // The last block to finish advances the epoch, so the records of this call can never be taken
    // for those of the next one and no per-call clearing is needed.
    if (p.carry_mode && tid == 0) {
        __threadfence();
        const unsigned done = atomicAdd(p.header + 1, 1u);
        if (done == gridDim.x - 1) {
            p.header[1] = 0;
            const unsigned e = ld_volatile_u32(p.header);
            p.header[0] = (e == 0xffffffffu) ? 1u : e + 1u;
        }
    }
}

}  // namespace rlcs
