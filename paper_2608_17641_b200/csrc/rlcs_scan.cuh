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
__host__ __device__ constexpr bool const_decay(int a) { return a != kVtrace && a != kRetrace && a != kAffineBwd && a != kAffineFwd; }

constexpr unsigned kDeviceTimeout = 7;   // RLCS_ERR_TIMEOUT
constexpr int kHeaderWords = 64;         // workspace header: 256 bytes
// header[0] = call counter (epoch), header[1] = finished-block counter, header[2] = status word

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
    float gamma;
    float decay;              // gamma*lambda | gamma | 1
    float aux;                // TD(lambda): gamma*(1-lambda); Retrace: lambda
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
// result = x (+) acc = (x.a + x.b*acc.a, x.b*acc.b)  (Eq. 2).  A zero beta selects x.a outright,
// so nothing from beyond a reset is ever touched.
__device__ __forceinline__ Pair apply(Pair x, Pair acc) {
    Pair r;
    r.a = (x.b != 0.f) ? fmaf(x.b, acc.a, x.a) : x.a;
    r.b = x.b * acc.b;
    return r;
}

__device__ __forceinline__ unsigned nonzero_bytes_to_bits(unsigned w) {
    // bit k of the result = (byte k of w != 0)
    unsigned nz = ((((w & 0x7f7f7f7fu) + 0x7f7f7f7fu) | w) >> 7) & 0x01010101u;
    return ((nz * 0x00204081u) >> 21) & 0xfu;
}

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

template <int ITEMS, bool VEC>
__device__ __forceinline__ unsigned load_mask(const uint8_t* __restrict__ p, long long i0, int nvalid) {
    unsigned m = 0;
    if (VEC && nvalid == ITEMS) {
        if constexpr (ITEMS == 4) {
            m = nonzero_bytes_to_bits(__ldcs(reinterpret_cast<const unsigned*>(p + i0)));
        } else if constexpr (ITEMS == 8) {
            uint2 v = __ldcs(reinterpret_cast<const uint2*>(p + i0));
            m = nonzero_bytes_to_bits(v.x) | (nonzero_bytes_to_bits(v.y) << 4);
        } else {
            static_assert(ITEMS == 16, "ITEMS must be 4, 8 or 16");
            uint4 v = __ldcs(reinterpret_cast<const uint4*>(p + i0));
            m = nonzero_bytes_to_bits(v.x) | (nonzero_bytes_to_bits(v.y) << 4) |
                (nonzero_bytes_to_bits(v.z) << 8) | (nonzero_bytes_to_bits(v.w) << 12);
        }
    } else {
#pragma unroll
        for (int j = 0; j < ITEMS; ++j)
            if (j < nvalid && __ldcs(p + i0 + j) != 0) m |= 1u << j;
    }
    return m;
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
__device__ __forceinline__ float lookback(const uint4* __restrict__ records, unsigned epoch, long long s,
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
        // fold lanes 0..min(z,31) in lane order (lane 0 = nearest tile)
        Pair cur = (lane <= z) ? p : Pair{0.f, 1.f};
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            Pair o;
            o.a = __shfl_down_sync(0xffffffffu, cur.a, d);
            o.b = __shfl_down_sync(0xffffffffu, cur.b, d);
            if (lane + d < 32) cur = apply(cur, o);
        }
        Pair w;
        w.a = __shfl_sync(0xffffffffu, cur.a, 0);
        w.b = __shfl_sync(0xffffffffu, cur.b, 0);
        acc = apply(acc, w);
        if (done) return acc.a;
        base -= 32;
    }
}

template <int ALGO, bool TRUNC, bool VEC, int THREADS, int ITEMS, int MIN_BLOCKS>
__global__ void __launch_bounds__(THREADS, MIN_BLOCKS) scan_kernel(const ScanParams p) {
    constexpr bool FWD = is_forward(ALGO);
    constexpr int NW = THREADS / 32;
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
        const unsigned q = (unsigned)i0 / p.T;
        n0 = q;
        t0 = (unsigned)i0 - q * p.T;
    } else {
        n0 = i0 / (long long)p.T;
        t0 = (unsigned)(i0 - n0 * (long long)p.T);
    }
    const unsigned Tm1 = p.T - 1;

    // ------------------------------------------------------------------ 1. loads (all issued up front)
    unsigned dmask = 0, tmask = 0;
    if constexpr (ALGO != kAffineBwd && ALGO != kAffineFwd) dmask = load_mask<ITEMS, VEC>(p.dones, i0, nvalid);
    if constexpr (TRUNC) tmask = load_mask<ITEMS, VEC>(p.truncs, i0, nvalid);

    float alpha[ITEMS];            // rewards | x | alpha, then alpha_t, then the first output
    load_f32<ITEMS, VEC>(p.f0, i0, nvalid, alpha);
    float x1[ITEMS];               // values | q_sa | beta
    if constexpr (ALGO != kDisc && ALGO != kElig && ALGO != kPrefix) load_f32<ITEMS, VEC>(p.f1, i0, nvalid, x1);
    float x2[ITEMS];               // expected_q
    if constexpr (ALGO == kRetrace) load_f32<ITEMS, VEC>(p.f2, i0, nvalid, x2);
    float x3[ITEMS];               // log_rhos
    if constexpr (ALGO == kVtrace || ALGO == kRetrace) load_f32<ITEMS, VEC>(p.f3, i0, nvalid, x3);

    // one-step halo beyond the thread's chunk, in time direction of the dependency
    float halo = 0.f, halo_lr = 0.f;
    unsigned halo_d = 0;
    if constexpr (!FWD && (has_values(ALGO) || ALGO == kRetrace)) {
        const float* src = (ALGO == kRetrace) ? p.f2 : p.f1;
        const bool edge = (lane == 31) && (rem > ITEMS);
        if (edge) halo = __ldg(src + i0 + ITEMS);
        if constexpr (ALGO == kRetrace) if (edge) halo_lr = __ldg(p.f3 + i0 + ITEMS);
    }
    if constexpr (ALGO == kElig || ALGO == kPrefix) {
        if (lane == 0 && i0 > 0 && rem > 0) halo_d = (__ldg(p.dones + i0 - 1) != 0);
    }

    // window-edge bootstrap of the first row edge inside the chunk (later edges only when T < ITEMS)
    float boot_first = 0.f;
    const unsigned to_edge = Tm1 - t0;           // steps from the chunk start to its row's last step
    if constexpr (!FWD && ALGO != kAffineBwd) {
        if (p.boot != nullptr && to_edge < (unsigned)nvalid) boot_first = __ldg(p.boot + n0);
    }

    // ------------------------------------------------------------------ 2. flags, sparse truncation values
    if constexpr (TRUNC) {
        tmask &= ~dmask;           // termination wins: trunc_bootstrap is not read there
    }
    float bv[ITEMS];
    if constexpr (TRUNC) {
#pragma unroll
        for (int j = 0; j < ITEMS; ++j) bv[j] = ((tmask >> j) & 1u) ? __ldg(p.trunc_boot + i0 + j) : 0.f;
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
    if constexpr (ALGO == kElig || (ALGO == kPrefix)) {
        const unsigned nb = __shfl_up_sync(FULL, (dmask >> (ITEMS - 1)) & 1u, 1);
        if (lane != 0) halo_d = nb;
    }

    // ------------------------------------------------------------------ 3. coefficients
    // contmask bit j: the recurrence continues from step j into its scan-order predecessor
    // (t+1 for backward scans, t-1 for forward scans).
    unsigned contmask = 0;
    float beta[ITEMS];             // only for algorithms with a per-step decay
    float grho[ITEMS];             // V-Trace: gamma*rho_t for the advantage epilogue
    {
        unsigned t = t0;
        long long n = n0;
#pragma unroll
        for (int j = 0; j < ITEMS; ++j) {
            const bool valid = j < nvalid;
            if constexpr (FWD) {
                const bool first = (t == 0);
                bool cont;
                if constexpr (ALGO == kAffineFwd) {
                    cont = !first;
                    beta[j] = (cont && valid) ? x1[j] : 0.f;
                } else {
                    const unsigned dprev = (j == 0) ? halo_d : ((dmask >> (j - 1)) & 1u);
                    const unsigned dsel = (ALGO == kPrefix && p.starts_at) ? ((dmask >> j) & 1u) : dprev;
                    cont = !first && !dsel;
                }
                if (cont && valid) contmask |= 1u << j;
            } else {
                const bool last = (t == Tm1);
                const bool term = (dmask >> j) & 1u;
                const bool trunc = TRUNC ? ((tmask >> j) & 1u) : false;
                const bool cont = valid && !term && !trunc && !last;
                if (cont) contmask |= 1u << j;
                if constexpr (ALGO == kAffineBwd) {
                    beta[j] = cont ? x1[j] : 0.f;
                } else {
                    float bootv = 0.f;
                    if (last && p.boot != nullptr && valid) bootv = ((unsigned)j == to_edge) ? boot_first : __ldg(p.boot + n);
                    // successor value of Section 3.2
                    float nextv = 0.f;
                    if constexpr (has_values(ALGO)) nextv = (j + 1 < ITEMS) ? x1[(j + 1) % ITEMS] : halo;
                    if constexpr (ALGO == kRetrace) nextv = (j + 1 < ITEMS) ? x2[(j + 1) % ITEMS] : halo;
                    float xn = last ? bootv : nextv;
                    if constexpr (TRUNC) xn = trunc ? bv[j] : xn;
                    xn = term ? 0.f : xn;
                    const float r = alpha[j];
                    if constexpr (ALGO == kGae) {
                        alpha[j] = fmaf(p.gamma, xn, r) - x1[j];
                    } else if constexpr (ALGO == kTdLambda) {
                        alpha[j] = fmaf(cont ? p.aux : p.gamma, xn, r);
                    } else if constexpr (ALGO == kDisc) {
                        alpha[j] = cont ? r : fmaf(p.gamma, xn, r);
                    } else if constexpr (ALGO == kVtrace) {
                        const float raw = expf(x3[j]);
                        const float rho = fminf(p.rho_bar, raw);
                        const float c = fminf(p.c_bar, raw);
                        alpha[j] = rho * (fmaf(p.gamma, xn, r) - x1[j]);
                        beta[j] = cont ? p.gamma * c : 0.f;
                        grho[j] = p.gamma * rho;
                    } else if constexpr (ALGO == kRetrace) {
                        alpha[j] = fmaf(p.gamma, xn, r) - x1[j];
                        const float lr_next = (j + 1 < ITEMS) ? x3[(j + 1) % ITEMS] : halo_lr;
                        beta[j] = cont ? p.gamma * (p.aux * fminf(p.c_bar, expf(lr_next))) : 0.f;
                    }
                    if (!valid) alpha[j] = 0.f;
                }
            }
            if (++t == p.T) { t = 0; ++n; }
        }
    }
    auto beta_of = [&](int j) -> float {
        if constexpr (const_decay(ALGO)) return ((contmask >> j) & 1u) ? p.decay : 0.f;
        else return beta[j];
    };

    // ------------------------------------------------------------------ 4. thread aggregate (serial combine, Eq. 2)
    Pair agg;
    if constexpr (FWD) {
        agg.a = alpha[0];
        agg.b = beta_of(0);
#pragma unroll
        for (int j = 1; j < ITEMS; ++j) {
            const float b = beta_of(j);
            agg.a = (b != 0.f) ? fmaf(b, agg.a, alpha[j]) : alpha[j];
            agg.b *= b;
        }
    } else {
        agg.a = alpha[ITEMS - 1];
        agg.b = beta_of(ITEMS - 1);
#pragma unroll
        for (int j = ITEMS - 2; j >= 0; --j) {
            const float b = beta_of(j);
            agg.a = (b != 0.f) ? fmaf(b, agg.a, alpha[j]) : alpha[j];
            agg.b *= b;
        }
    }

    // ------------------------------------------------------------------ 5. warp scan in scan order
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

    // ------------------------------------------------------------------ 6. block carry through shared memory
    const int wrank = FWD ? warp : NW - 1 - warp;
    if (rank == 31) s_agg[wrank] = incl;
    if (wrank == 0 && rank == 0) {
        // the tile's first step in scan order: does the recurrence enter the tile from outside?
        const int jfirst = FWD ? 0 : ITEMS - 1;
        s_need = (int)((contmask >> jfirst) & 1u);
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

    // ------------------------------------------------------------------ 7. carry between thread blocks
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
    float prev = (before.b != 0.f) ? fmaf(before.b, carry_in, before.a) : before.a;

    // ------------------------------------------------------------------ 8. replay, epilogue, store
    float out1v[ITEMS];
    if constexpr (FWD) {
#pragma unroll
        for (int j = 0; j < ITEMS; ++j) {
            const float b = beta_of(j);
            prev = (b != 0.f) ? fmaf(b, prev, alpha[j]) : alpha[j];
            alpha[j] = prev;
        }
    } else {
#pragma unroll
        for (int j = ITEMS - 1; j >= 0; --j) {
            const float b = beta_of(j);
            const float d = (b != 0.f) ? fmaf(b, prev, alpha[j]) : alpha[j];
            if constexpr (ALGO == kGae) {
                alpha[j] = d;
                out1v[j] = d + x1[j];
            } else if constexpr (ALGO == kVtrace) {
                // A_t = rho_t (r_t + gamma v_{t+1} - V_t) = alpha_t + gamma rho_t Delta_{t+1} where the
                // recurrence continues (v_{t+1} = V_{t+1} + Delta_{t+1}), alpha_t elsewhere.
                out1v[j] = ((contmask >> j) & 1u) ? fmaf(grho[j], prev, alpha[j]) : alpha[j];
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

    // ------------------------------------------------------------------ 9. close the call (carry mode)
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
