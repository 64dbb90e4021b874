// Fused segmented affine scan over the flattened [N*T] rollout array (sm_100a).
//
// The row-major [N, T] tensors are treated as one contiguous array of N*T steps that is cut into
// fixed tiles of THREADS*ITEMS steps; a row edge is simply one more reset.  Per tile a thread block
//   1. brings ITEMS consecutive steps of each input per thread on chip, plus a one-step halo of the
//      successor value;
//   2. builds (alpha_t, beta_t) of Table 1 in registers, with the boundary rules of Section 3.2
//      and the window-edge carry folded into alpha, so that every row scans with carry 0;
//   3. folds each thread's ITEMS pairs serially with the combine of Eq. 2, scans the per-thread
//      aggregates with warp shuffles, and the per-warp aggregates through shared memory;
//   4. if the tile is entered in the middle of an episode, obtains the carry from the preceding
//      tiles (in scan order) by a bounded, deterministic look-back over published tile aggregates;
//   5. replays the recurrence over its ITEMS steps from the carry, applies the epilogue
//      (returns = A + V, V-Trace targets and advantages, Retrace targets) and stores once.
// Backward algorithms scan from high addresses to low ones: scan-order tile s is address tile
// num_tiles-1-s, so a block only ever waits on tiles with a smaller scan-order index.
//
// Two kernels share this per-tile code:
//   scan_kernel_tma  persistent thread blocks (all co-resident); each walks tiles s, s+G, s+2G, ...
//                    and keeps a ring of STAGES tiles in flight: one elected thread issues 1-D bulk
//                    copies (cp.async.bulk into its own block's shared memory, no tensor map: tiles of the flat array are
//                    contiguous) that complete on an mbarrier per stage.  Needs 16-byte aligned
//                    pointers; the ragged last tile(s) are loaded with plain loads.
//   scan_kernel      one tile per thread block, plain (vector or element-wise) global loads; used
//                    for unaligned pointers and as the cross-check in the tests.
//
// The per-step code is branch-free: flags stay packed as mask bytes (4 steps per 32-bit word), a
// reset is a beta of exactly 0, successor values at resets are selected (never multiplied), and
// the rare cases -- a row edge inside a thread's chunk, the ragged last chunk, rows shorter than a
// chunk -- patch the packed words in short side paths.
#pragma once

#include <cooperative_groups.h>
#include <cuda_runtime.h>
#include <stdint.h>

// Element type of the float tensors in global memory.  A translation unit that defines
// RLCS_IO_BF16 before including this header gets the same kernels with bfloat16 tensors (inputs
// widened to fp32 on load -- exact -- and all arithmetic in fp32 registers, outputs rounded to
// nearest-even on store) in a namespace of their own, so that both builds link into one library.
#ifdef RLCS_IO_BF16
#include <cuda_bf16.h>
#define RLCS_NS rlcs_bf16
namespace RLCS_NS {
using io_t = __nv_bfloat16;
constexpr bool kIoBf16 = true;
}
#else
#define RLCS_NS rlcs
namespace RLCS_NS {
using io_t = float;
constexpr bool kIoBf16 = false;
}
#endif

namespace RLCS_NS {

enum Algo : int {
    kGae = 0, kTdLambda = 1, kDisc = 2, kVtrace = 3, kRetrace = 4, kElig = 5, kPrefix = 6,
    kAffineBwd = 7, kAffineFwd = 8,
    kGaeStats = 9,    // GAE that also leaves per-tile sums of A and of its squared deviations (for advantage normalisation)
    kRetraceProbs = 10, // Retrace(lambda) from [N,T,A] Q-values and action probabilities
    // Observation-skip masking (Section 9.2): masked steps are transparent.  Two scans:
    kFillSkip = 11,     // W_t = V_t at unmasked steps, the successor's W (or the flag's successor value) at masked ones
    kGaeSkip = 12       // GAE on rewards and W with alpha_t = 0, beta_t = 1 at masked steps
};

__host__ __device__ constexpr bool is_forward(int a) { return a == kElig || a == kPrefix || a == kAffineFwd; }
__host__ __device__ constexpr bool is_gae(int a) { return a == kGae || a == kGaeStats || a == kGaeSkip; }
__host__ __device__ constexpr bool uses_skip(int a) { return a == kFillSkip || a == kGaeSkip; }
__host__ __device__ constexpr bool has_values(int a) { return is_gae(a) || a == kTdLambda || a == kVtrace; }
__host__ __device__ constexpr bool is_affine(int a) { return a == kAffineBwd || a == kAffineFwd; }
__host__ __device__ constexpr bool is_retrace(int a) { return a == kRetrace || a == kRetraceProbs; }
__host__ __device__ constexpr bool const_decay(int a) { return a != kVtrace && !is_retrace(a) && !is_affine(a) && !uses_skip(a); }
// a float input is read one step beyond the tile (successor value)
__host__ __device__ constexpr bool float_halo(int a) { return has_values(a) || is_retrace(a); }
__host__ __device__ constexpr bool uses_f1(int a) { return a != kDisc && a != kElig && a != kPrefix && a != kFillSkip; }
__host__ __device__ constexpr bool uses_f2(int a) { return a == kRetrace; }
__host__ __device__ constexpr bool uses_f3(int a) { return a == kVtrace || a == kRetrace; }
__host__ __device__ constexpr bool uses_dones(int a) { return !is_affine(a); }

constexpr unsigned kDeviceTimeout = 7;   // RLCS_ERR_TIMEOUT
constexpr int kHeaderWords = 64;         // workspace header: 256 bytes
// header[0] = call counter (epoch), header[1] = finished-block counter, header[2] = status word

// Division of a 32-bit index by the invariant row length T (Granlund-Montgomery, round-up form):
// q = (hi + ((n - hi) >> sh1)) >> sh2 with hi = umulhi(mul, n).  Exact for every n < 2^32, T >= 1.
struct FastDiv {
    unsigned mul, sh1, sh2;
};

struct ScanParams {
    const io_t* f0;           // rewards | x | alpha
    const io_t* f1;           // values | q_sa | beta
    const io_t* f2;           // expected_q
    const io_t* f3;           // log_rhos
    const float* pi;          // kRetraceProbs: target-policy probabilities [N,T,A]  (f1 = Q-values [N,T,A])
    const float* mu;          // kRetraceProbs: behaviour-policy probabilities [N,T,A]
    const int* actions;       // kRetraceProbs: actions taken [N,T]
    int A;                    // kRetraceProbs: number of actions
    const uint8_t* dones;
    const uint8_t* truncs;
    const uint8_t* skip;      // kFillSkip, kGaeSkip: non-zero = masked step
    const io_t* trunc_boot;   // [N,T]
    const io_t* boot;         // [N] or nullptr
    io_t* out0;
    io_t* out1;               // second output or nullptr
    io_t* out2;               // scan_kernel_gae_skip: the filled values W
    float* stats;             // kGaeStats: per scan-order tile {sum A, sum (A - tile mean)^2}
    long long total;          // N*T
    long long num_tiles;
    unsigned tile_steps;      // steps a thread block covers: THREADS*ITEMS, or a whole number of rows that is a little
                              // less (row-aligned tiling: the last few threads idle, but no row straddles a tile)
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
    int cluster;              // > 1: rows are exactly this many tiles long, one thread-block cluster per row
    int row_blocks;           // != 0: one thread block per row walks the row's tiles in scan order (scan_kernel_rows)
    unsigned* header;         // workspace header (carry mode) or nullptr
    unsigned* status;         // device status word, or nullptr when there is no workspace
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

// ------------------------------------------------------------------------------------------ programmatic dependent launch
// The kernels are launched with programmatic stream serialisation: the blocks of a launch may be
// placed on the SMs while the previous kernel of the stream is still draining, so that launch
// latency and block set-up overlap that kernel's tail.  grid_dependency_wait() returns once the
// previous kernel has completed and its writes are visible; NOTHING in global memory -- caller
// tensors, the workspace header, tile records -- is read or written before it.
// grid_dependency_launch() tells the scheduler that the next launch's blocks may be placed; it is
// given first thing, because a later kernel still waits for this one's completion at its own
// grid_dependency_wait().  Both are no-ops for a launch without the attribute.
__device__ __forceinline__ void grid_dependency_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// ------------------------------------------------------------------------------------------ global loads / stores
// 256-bit global accesses (sm_100): one instruction moves a thread's 8 consecutive fp32 values, so a
// warp touches 1 KiB of whole 32-byte sectors per instruction.  32-byte aligned addresses only.
__device__ __forceinline__ void ldg_v8(const float* p, float* x) {
    asm volatile("ld.global.nc.L1::no_allocate.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=f"(x[0]), "=f"(x[1]), "=f"(x[2]), "=f"(x[3]), "=f"(x[4]), "=f"(x[5]), "=f"(x[6]), "=f"(x[7])
                 : "l"(p));
}
__device__ __forceinline__ void stg_v8(float* p, const float* x) {
    asm volatile("st.global.cs.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 :: "l"(p), "f"(x[0]), "f"(x[1]), "f"(x[2]), "f"(x[3]), "f"(x[4]), "f"(x[5]), "f"(x[6]), "f"(x[7])
                 : "memory");
}
// Load *p if pred, else keep 0: a predicated load instead of a branch around a load.
__device__ __forceinline__ float ldg_if(const float* p, bool pred) {
    float v = 0.f;
    asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.u32 q, %2, 0;\n\t@q ld.global.nc.f32 %0, [%1];\n\t}"
                 : "+f"(v) : "l"(p), "r"((unsigned)pred));
    return v;
}

// ALLORNONE (with VEC): the chunk is either whole or empty (an idle thread of a row-aligned tile),
// so there is no element-wise path to compile.
template <int ITEMS, bool VEC, bool ALLORNONE = false>
__device__ __forceinline__ void load_f32(const float* __restrict__ p, long long i0, int nvalid, float (&x)[ITEMS]) {
    if constexpr (VEC && ALLORNONE) {
        if (nvalid != ITEMS) {
#pragma unroll
            for (int j = 0; j < ITEMS; ++j) x[j] = 0.f;
            return;
        }
    }
    if (VEC && nvalid == ITEMS) {
        if constexpr (ITEMS % 8 == 0) {
#pragma unroll
            for (int k = 0; k < ITEMS / 8; ++k) ldg_v8(p + i0 + 8 * k, &x[8 * k]);
        } else {
            const float4* q = reinterpret_cast<const float4*>(p + i0);
#pragma unroll
            for (int k = 0; k < ITEMS / 4; ++k) {
                float4 v = __ldcs(q + k);
                x[4 * k + 0] = v.x; x[4 * k + 1] = v.y; x[4 * k + 2] = v.z; x[4 * k + 3] = v.w;
            }
        }
    } else {
#pragma unroll
        for (int j = 0; j < ITEMS; ++j) x[j] = (j < nvalid) ? __ldcs(p + i0 + j) : 0.f;
    }
}

// Mask bytes of ITEMS consecutive steps, packed 4 per word (byte j%4 of word j/4), values as stored
// (any non-zero byte = true).
template <int ITEMS, bool VEC, bool ALLORNONE = false>
__device__ __forceinline__ void load_mask(const uint8_t* __restrict__ p, long long i0, int nvalid, unsigned (&w)[ITEMS / 4]) {
    if constexpr (VEC && ALLORNONE) {
        if (nvalid != ITEMS) {
#pragma unroll
            for (int k = 0; k < ITEMS / 4; ++k) w[k] = 0;
            return;
        }
    }
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
        if constexpr (ITEMS % 8 == 0) {
#pragma unroll
            for (int k = 0; k < ITEMS / 8; ++k) stg_v8(p + i0 + 8 * k, &x[8 * k]);
        } else {
            float4* q = reinterpret_cast<float4*>(p + i0);
#pragma unroll
            for (int k = 0; k < ITEMS / 4; ++k)
                __stcs(q + k, make_float4(x[4 * k + 0], x[4 * k + 1], x[4 * k + 2], x[4 * k + 3]));
        }
    } else {
#pragma unroll
        for (int j = 0; j < ITEMS; ++j)
            if (j < nvalid) __stcs(p + i0 + j, x[j]);
    }
}

#ifdef RLCS_IO_BF16
// bfloat16 tensors: a 32-bit word holds two consecutive elements (low half first); widening is a
// shift or a mask, narrowing is cvt.rn.bf16x2.f32 (round to nearest even).
__device__ __forceinline__ void widen2(unsigned w, float& lo, float& hi) {
    lo = __uint_as_float(w << 16);
    hi = __uint_as_float(w & 0xffff0000u);
}
__device__ __forceinline__ unsigned narrow2(float lo, float hi) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const unsigned*>(&h);
}
__device__ __forceinline__ float ld_io(const io_t* p) {
    return __uint_as_float((unsigned)__ldg(reinterpret_cast<const unsigned short*>(p)) << 16);
}
__device__ __forceinline__ float ldg_if(const io_t* p, bool pred) {
    unsigned short v = 0;
    asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.u32 q, %2, 0;\n\t@q ld.global.nc.u16 %0, [%1];\n\t}"
                 : "+h"(v) : "l"(p), "r"((unsigned)pred));
    return __uint_as_float((unsigned)v << 16);
}

template <int ITEMS, bool VEC, bool ALLORNONE = false>
__device__ __forceinline__ void load_f32(const io_t* __restrict__ p, long long i0, int nvalid, float (&x)[ITEMS]) {
    if constexpr (VEC && ALLORNONE) {
        if (nvalid != ITEMS) {
#pragma unroll
            for (int j = 0; j < ITEMS; ++j) x[j] = 0.f;
            return;
        }
    }
    if (VEC && nvalid == ITEMS) {
        unsigned w[ITEMS / 2];
        if constexpr (ITEMS == 16) {
            asm volatile("ld.global.nc.L1::no_allocate.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                         : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]), "=r"(w[4]), "=r"(w[5]), "=r"(w[6]), "=r"(w[7])
                         : "l"(p + i0));
        } else if constexpr (ITEMS == 8) {
            const uint4 v = __ldcs(reinterpret_cast<const uint4*>(p + i0));
            w[0] = v.x; w[1] = v.y; w[2] = v.z; w[3] = v.w;
        } else {
            static_assert(ITEMS == 4, "ITEMS must be 4, 8 or 16");
            const uint2 v = __ldcs(reinterpret_cast<const uint2*>(p + i0));
            w[0] = v.x; w[1] = v.y;
        }
#pragma unroll
        for (int k = 0; k < ITEMS / 2; ++k) widen2(w[k], x[2 * k], x[2 * k + 1]);
    } else {
        const unsigned short* q = reinterpret_cast<const unsigned short*>(p) + i0;
#pragma unroll
        for (int j = 0; j < ITEMS; ++j) x[j] = (j < nvalid) ? __uint_as_float((unsigned)__ldcs(q + j) << 16) : 0.f;
    }
}

template <int ITEMS, bool VEC>
__device__ __forceinline__ void store_f32(io_t* __restrict__ p, long long i0, int nvalid, const float (&x)[ITEMS]) {
    if (VEC && nvalid == ITEMS) {
        unsigned w[ITEMS / 2];
#pragma unroll
        for (int k = 0; k < ITEMS / 2; ++k) w[k] = narrow2(x[2 * k], x[2 * k + 1]);
        if constexpr (ITEMS == 16) {
            asm volatile("st.global.cs.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                         :: "l"(p + i0), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7])
                         : "memory");
        } else if constexpr (ITEMS == 8) {
            __stcs(reinterpret_cast<uint4*>(p + i0), make_uint4(w[0], w[1], w[2], w[3]));
        } else {
            __stcs(reinterpret_cast<uint2*>(p + i0), make_uint2(w[0], w[1]));
        }
    } else {
        unsigned short* q = reinterpret_cast<unsigned short*>(p) + i0;
#pragma unroll
        for (int j = 0; j < ITEMS; ++j)
            if (j < nvalid) __stcs(q + j, (unsigned short)(narrow2(x[j], 0.f) & 0xffffu));
    }
}
#else
__device__ __forceinline__ float ld_io(const io_t* p) { return __ldg(p); }
#endif

// ------------------------------------------------------------------------------------------ shared-memory reads
template <int ITEMS>
__device__ __forceinline__ void lds_f32(const float* s, float (&x)[ITEMS]) {   // s is 16-byte aligned
    const float4* q = reinterpret_cast<const float4*>(s);
#pragma unroll
    for (int k = 0; k < ITEMS / 4; ++k) {
        float4 v = q[k];
        x[4 * k + 0] = v.x; x[4 * k + 1] = v.y; x[4 * k + 2] = v.z; x[4 * k + 3] = v.w;
    }
}
template <int ITEMS>
__device__ __forceinline__ void lds_mask(const uint8_t* s, unsigned (&w)[ITEMS / 4]) {   // s is ITEMS-byte aligned
    if constexpr (ITEMS == 4) {
        w[0] = *reinterpret_cast<const unsigned*>(s);
    } else if constexpr (ITEMS == 8) {
        uint2 v = *reinterpret_cast<const uint2*>(s);
        w[0] = v.x; w[1] = v.y;
    } else {
        uint4 v = *reinterpret_cast<const uint4*>(s);
        w[0] = v.x; w[1] = v.y; w[2] = v.z; w[3] = v.w;
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
// (Pure shift arithmetic on purpose: a select between array elements would let the compiler index
// the array dynamically and move the whole chunk to local memory.)
template <int W>
__device__ __forceinline__ bool test_byte_dyn(const unsigned (&w)[W], unsigned j) {
    static_assert(W == 1 || W == 2 || W == 4, "unsupported chunk width");
    if constexpr (W == 1) {
        return ((w[0] >> (j * 8u)) & 0xffu) != 0;
    } else if constexpr (W == 2) {
        const unsigned long long v = ((unsigned long long)w[1] << 32) | w[0];
        return ((v >> (j * 8u)) & 0xffull) != 0;
    } else {
        const unsigned long long lo = ((unsigned long long)w[1] << 32) | w[0];
        const unsigned long long hi = ((unsigned long long)w[3] << 32) | w[2];
        const unsigned long long m = 0ull - (unsigned long long)((j >> 3) & 1u);      // all ones for the upper half
        const unsigned long long v = (hi & m) | (lo & ~m);
        return ((v >> ((j & 7u) * 8u)) & 0xffull) != 0;
    }
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

// A block signs off from the carry protocol of this call once it has published its last record and
// finished its last look-back: from then on it neither reads the epoch nor polls records.  The last
// block to sign off advances the epoch, so the records of this call can never be taken for those
// of the next one and no per-call clearing is needed.  (No fence: nothing but the protocol words
// depends on it, and the next call starts only after this kernel has ended.)  Signing off before
// the stores keeps this round trip off the tail of the kernel.
__device__ __forceinline__ void sign_off(const ScanParams& p) {
    if (threadIdx.x == 0) {
        const unsigned done = atomicAdd(p.header + 1, 1u);
        if (done == gridDim.x - 1) {
            p.header[1] = 0;
            const unsigned e = ld_volatile_u32(p.header);
            p.header[0] = (e == 0xffffffffu) ? 256u : e + 1u;      // never 0..255 (see rlcs_workspace_init)
        }
    }
}

// ------------------------------------------------------------------------------------------ one thread's part of a tile
// Flags and geometry of a thread's ITEMS consecutive steps: everything the coefficient stage needs
// besides the float inputs.  The persistent kernel fetches this one tile ahead.
template <int ALGO, bool TRUNC, int ITEMS>
struct Chunk {
    static constexpr int W = ITEMS / 4;
    unsigned edge;           // offset of the first row edge at or after the chunk start (see locate)
    int nvalid;              // steps of the chunk inside the array
    unsigned dw[W], tw[W];   // dones / truncs mask bytes
    unsigned kw[uses_skip(ALGO) ? W : 1];   // skip mask bytes (observation-skip masking)
    unsigned halo_d;         // forward scans: dones byte of the step before the chunk
    float ov[ITEMS];         // successor value where the recurrence is severed (0 | trunc_bootstrap | bootstrap)
    float boot_first;        // window-edge bootstrap of the row whose edge lies in the chunk
};

// The float inputs of the same steps.
template <int ITEMS>
struct Vals {
    float a[ITEMS];          // rewards | x | alpha; then alpha_t; then the first output
    float x1[ITEMS];         // values | q_sa | beta
    float x2[ITEMS];         // expected_q
    float x3[ITEMS];         // log_rhos
    float halo, halo_lr;     // successor-side neighbour of the chunk's last step (values | expected_q, log_rhos)
};

// Row / timestep of flat index i0, and the chunk offset of the first row edge: for backward scans
// the row's last step (offset T-1-t0); for forward scans the next row's first step (offset T-t0, or
// 0 when the chunk itself starts a row).
template <int ALGO, bool TRUNC, int ITEMS>
__device__ __forceinline__ long long locate(Chunk<ALGO, TRUNC, ITEMS>& c, const ScanParams& p, long long i0, long long end) {
    const long long rem = end - i0;            // `end`: the array's end, or this tile's end when it comes first
    c.nvalid = rem >= ITEMS ? ITEMS : (rem > 0 ? (int)rem : 0);
    unsigned t0;
    long long n0;
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
    c.edge = is_forward(ALGO) ? (t0 == 0 ? 0u : p.T - t0) : (p.T - 1 - t0);
    return n0;               // the row of step i0
}
template <int ALGO, bool TRUNC, int ITEMS>
__device__ __forceinline__ long long locate(Chunk<ALGO, TRUNC, ITEMS>& c, const ScanParams& p, long long i0) {
    return locate(c, p, i0, p.total);
}

// Window-edge bootstrap of the first row edge inside the chunk (plain load, issued early).
template <int ALGO, bool TRUNC, int ITEMS>
__device__ __forceinline__ void issue_boot(Chunk<ALGO, TRUNC, ITEMS>& c, const ScanParams& p, long long n0) {
    c.boot_first = 0.f;
    if constexpr (!is_forward(ALGO) && !is_affine(ALGO)) {
        c.boot_first = ldg_if(p.boot + n0, p.boot != nullptr && c.edge < (unsigned)c.nvalid);
    }
}

// Mask bytes from global memory; forward scans also need the dones byte just before the chunk.
// IDLE (with FULL): row-aligned tiling -- every thread of the block has a whole chunk or none at all.
template <int ALGO, bool TRUNC, int ITEMS, bool VEC, bool FULL = false, bool IDLE = false>
__device__ __forceinline__ void load_flags_global(Chunk<ALGO, TRUNC, ITEMS>& c, const ScanParams& p, long long i0, int lane) {
    constexpr int W = ITEMS / 4;
    const int nvalid = (FULL && !IDLE) ? ITEMS : c.nvalid;
#pragma unroll
    for (int k = 0; k < W; ++k) { c.dw[k] = 0; c.tw[k] = 0; }
    c.halo_d = 0;
    if constexpr (ALGO == kElig || ALGO == kPrefix) {
        if (lane == 0 && i0 > 0 && nvalid > 0) c.halo_d = __ldg(p.dones + i0 - 1);
    }
    if constexpr (uses_dones(ALGO)) load_mask<ITEMS, VEC, IDLE>(p.dones, i0, nvalid, c.dw);
    if constexpr (TRUNC) load_mask<ITEMS, VEC, IDLE>(p.truncs, i0, nvalid, c.tw);
    if constexpr (uses_skip(ALGO)) load_mask<ITEMS, VEC, IDLE>(p.skip, i0, nvalid, c.kw);
    if constexpr (ALGO == kElig || ALGO == kPrefix) {
        const unsigned nb = __shfl_up_sync(0xffffffffu, c.dw[W - 1] >> 24, 1);
        if (lane != 0) c.halo_d = nb;
    }
}

// Sparse truncation continuation values: only where truncs is set and dones is not.
// SECTORS (fp32 tensors, whole chunk inside the array, 32-byte aligned): one predicated 256-bit load
// per 32-byte sector that holds a needed value instead of one predicated scalar load per step -- the
// same sectors cross DRAM, in an eighth of the requests.
__device__ __forceinline__ unsigned nonzero_bytes(unsigned w) {      // 0x80 in every byte of w that is not zero
    return (((w & 0x7f7f7f7fu) + 0x7f7f7f7fu) | w) & 0x80808080u;
}
template <int ALGO, bool TRUNC, int ITEMS, bool SECTORS = false>
__device__ __forceinline__ void issue_trunc_values(Chunk<ALGO, TRUNC, ITEMS>& c, const ScanParams& p, long long i0) {
#pragma unroll
    for (int j = 0; j < ITEMS; ++j) c.ov[j] = 0.f;
    if constexpr (TRUNC) {
        // (TD(lambda) keeps the per-step form: it runs at a 64-register cap where the sector form spills
        // more -- measured 72.5 -> 73.9 us at 16384 x 2048, against 57.2 -> 55.6 for the discounted return and
        // 10.7 -> 10.2 / 18.6 -> 17.8 us for V-trace at 4096 x 512 / 4096 x 1024)
        if constexpr (SECTORS && !kIoBf16 && ITEMS % 8 == 0 && ALGO != kTdLambda) {
#pragma unroll
            for (int k = 0; k < ITEMS / 8; ++k) {
                const unsigned n0 = nonzero_bytes(c.tw[2 * k]) & ~nonzero_bytes(c.dw[2 * k]);
                const unsigned n1 = nonzero_bytes(c.tw[2 * k + 1]) & ~nonzero_bytes(c.dw[2 * k + 1]);
                float x[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
                asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.u32 q, %9, 0;\n\t"
                             "@q ld.global.nc.L1::no_allocate.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];\n\t}"
                             : "+f"(x[0]), "+f"(x[1]), "+f"(x[2]), "+f"(x[3]), "+f"(x[4]), "+f"(x[5]), "+f"(x[6]), "+f"(x[7])
                             : "l"(reinterpret_cast<const float*>(p.trunc_boot) + i0 + 8 * k), "r"(n0 | n1));
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const unsigned bit = 0x80u << (8 * (j % 4));
                    c.ov[8 * k + j] = (((j < 4 ? n0 : n1) & bit) != 0) ? x[j] : 0.f;
                }
            }
        } else if constexpr (SECTORS && kIoBf16 && ITEMS == 16 && ALGO != kTdLambda) {
            // bfloat16 tensors: a thread's 16 steps are exactly one 32-byte sector
            unsigned need[4], any = 0;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                need[k] = nonzero_bytes(c.tw[k]) & ~nonzero_bytes(c.dw[k]);
                any |= need[k];
            }
            unsigned w[8] = {0, 0, 0, 0, 0, 0, 0, 0};
            asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.u32 q, %9, 0;\n\t"
                         "@q ld.global.nc.L1::no_allocate.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];\n\t}"
                         : "+r"(w[0]), "+r"(w[1]), "+r"(w[2]), "+r"(w[3]), "+r"(w[4]), "+r"(w[5]), "+r"(w[6]), "+r"(w[7])
                         : "l"(p.trunc_boot + i0), "r"(any));
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                const float x = __uint_as_float((j & 1) ? (w[j / 2] & 0xffff0000u) : (w[j / 2] << 16));
                c.ov[j] = ((need[j / 4] & (0x80u << (8 * (j % 4)))) != 0) ? x : 0.f;
            }
        } else {
#pragma unroll
            for (int j = 0; j < ITEMS; ++j)
                c.ov[j] = ldg_if(p.trunc_boot + i0 + j, test_byte(c.tw, j) && !test_byte(c.dw, j));
        }
    }
}

// Float inputs from global memory, with the one-step halo (lane 31 loads it, the others take
// their neighbour's first element).
template <int ALGO, bool TRUNC, int ITEMS, bool VEC, bool FULL = false, bool IDLE = false>
__device__ __forceinline__ void load_values_global(const Chunk<ALGO, TRUNC, ITEMS>& c, Vals<ITEMS>& v, const ScanParams& p, long long i0, int lane) {
    const int nvalid = (FULL && !IDLE) ? ITEMS : c.nvalid;
    load_f32<ITEMS, VEC, IDLE>(p.f0, i0, nvalid, v.a);
    if constexpr (uses_f1(ALGO)) load_f32<ITEMS, VEC, IDLE>(p.f1, i0, nvalid, v.x1);
    if constexpr (uses_f2(ALGO)) load_f32<ITEMS, VEC, IDLE>(p.f2, i0, nvalid, v.x2);
    if constexpr (uses_f3(ALGO)) load_f32<ITEMS, VEC, IDLE>(p.f3, i0, nvalid, v.x3);
    v.halo = 0.f;
    v.halo_lr = 0.f;
    if constexpr (float_halo(ALGO)) {
        const io_t* src = (ALGO == kRetrace) ? p.f2 : p.f1;
        const bool edge_lane = (lane == 31) && (p.total - i0 > ITEMS);
        v.halo = ldg_if(src + i0 + ITEMS, edge_lane);
        if constexpr (ALGO == kRetrace) v.halo_lr = ldg_if(p.f3 + i0 + ITEMS, edge_lane);
        const float first = (ALGO == kRetrace) ? v.x2[0] : v.x1[0];
        const float nb = __shfl_down_sync(0xffffffffu, first, 1);
        if (lane != 31) v.halo = nb;
        if constexpr (ALGO == kRetrace) {
            const float nl = __shfl_down_sync(0xffffffffu, v.x3[0], 1);
            if (lane != 31) v.halo_lr = nl;
        }
    }
}

#ifndef RLCS_IO_BF16   // the [N,T,A] form stays fp32
// Retrace from the [N,T,A] tensors: per step, Q(s_t,a_t), E_pi Q(s_t,.) = sum_a pi(a|s_t) Q(s_t,a) and the
// importance ratio pi(a_t|s_t)/mu(a_t|s_t) are formed here from one dense read of the Q and pi rows
// and three gathers, and only those three scalars per step stay in registers -- the tile never
// holds whole [T, A] slabs, so the register need does not grow with T.  AV = A when known at
// compile time (vector loads), 0 = any A.  Actions outside [0, A) are clamped (memory safety only).
template <int AV>
__device__ __forceinline__ void probs_step(const ScanParams& p, long long i, bool active, float& q_sa, float& eq, float& ratio) {
    q_sa = 0.f; eq = 0.f; ratio = 0.f;
    if (!active) return;
    const int A = AV > 0 ? AV : p.A;
    const float* __restrict__ qrow = p.f1 + i * A;
    const float* __restrict__ prow = p.pi + i * A;
    int act = __ldg(p.actions + i);
    act = act < 0 ? 0 : (act >= A ? A - 1 : act);
    float e = 0.f;
    if constexpr (AV > 0 && AV % 8 == 0) {
#pragma unroll
        for (int k = 0; k < AV / 8; ++k) {
            float a[8], b[8];
            ldg_v8(qrow + 8 * k, a);
            ldg_v8(prow + 8 * k, b);
#pragma unroll
            for (int x = 0; x < 8; ++x) e = fmaf(b[x], a[x], e);
        }
    } else {
        for (int a = 0; a < A; ++a) e = fmaf(__ldcs(prow + a), __ldcs(qrow + a), e);
    }
    eq = e;
    q_sa = __ldg(qrow + act);
    ratio = __ldg(prow + act) / __ldg(p.mu + i * A + act);
}

// value of row[act] for a row held in registers (A small and known): a select chain, no second trip to memory
template <int A>
__device__ __forceinline__ float pick(const float* row, int act) {
    float v = row[0];
#pragma unroll
    for (int a = 1; a < A; ++a) v = (act == a) ? row[a] : v;
    return v;
}

template <int ALGO, bool TRUNC, int ITEMS, int AV>
__device__ __forceinline__ void load_values_probs(const Chunk<ALGO, TRUNC, ITEMS>& c, Vals<ITEMS>& v, const ScanParams& p,
                                                  long long i0, int lane, int nvalid) {
    load_f32<ITEMS, false>(p.f0, i0, nvalid, v.a);               // rewards (element-wise: this kernel is bound by the 3-D reads)
    if constexpr (AV == 4 || AV == 8) {
        // Rows of 16 or 32 bytes: a gathered mu(a_t|s_t) would touch every 32-byte sector of mu anyway,
        // so all three rows are read densely with 256-bit loads (no load depends on the action) and
        // Q(s_t,a_t), pi(a_t|s_t), mu(a_t|s_t) are picked from registers.  Needs full chunks; the ragged
        // tail falls through to the step-by-step path.
        if (nvalid == ITEMS) {
            constexpr int ROWS = 8 / AV;                         // rows per 256-bit load
            int act[ITEMS];
#pragma unroll
            for (int j = 0; j < ITEMS; ++j) {
                const int a = __ldg(p.actions + i0 + j);
                act[j] = a < 0 ? 0 : (a >= AV ? AV - 1 : a);
            }
#pragma unroll
            for (int j = 0; j < ITEMS; j += ROWS) {
                float q[8], pr[8], m[8];
                ldg_v8(p.f1 + (i0 + j) * AV, q);
                ldg_v8(p.pi + (i0 + j) * AV, pr);
                ldg_v8(p.mu + (i0 + j) * AV, m);
#pragma unroll
                for (int r = 0; r < ROWS; ++r) {
                    float e = 0.f;
#pragma unroll
                    for (int a = 0; a < AV; ++a) e = fmaf(pr[r * AV + a], q[r * AV + a], e);
                    v.x2[j + r] = e;
                    v.x1[j + r] = pick<AV>(q + r * AV, act[j + r]);
                    v.x3[j + r] = pick<AV>(pr + r * AV, act[j + r]) / pick<AV>(m + r * AV, act[j + r]);
                }
            }
        } else {
#pragma unroll
            for (int j = 0; j < ITEMS; ++j) probs_step<0>(p, i0 + j, j < nvalid, v.x1[j], v.x2[j], v.x3[j]);
        }
    } else {
#pragma unroll
        for (int j = 0; j < ITEMS; ++j) probs_step<AV>(p, i0 + j, j < nvalid, v.x1[j], v.x2[j], v.x3[j]);
    }
    // successor-side neighbour: the next thread's first step, or one more step from memory at the warp edge
    float hq, heq = 0.f, hr = 0.f;
    const bool edge_lane = (lane == 31) && (p.total - i0 > ITEMS);
    if (edge_lane) probs_step<0>(p, i0 + ITEMS, true, hq, heq, hr);
    const float nb = __shfl_down_sync(0xffffffffu, v.x2[0], 1);
    const float nr = __shfl_down_sync(0xffffffffu, v.x3[0], 1);
    v.halo = (lane != 31) ? nb : heq;
    v.halo_lr = (lane != 31) ? nr : hr;
}

#endif  // !RLCS_IO_BF16

// Shared-memory scratch of the block-level scan; double-buffered by tile parity in the persistent
// kernel so that one barrier per tile suffices.
template <int NW>
struct ScanSmem {
    Pair agg[2][NW];     // warp aggregates, indexed by the warp's rank in scan order
    float carry[2];      // tile carry-in
    int need[2];         // the tile is entered mid-episode
    Pair cl_agg;         // cluster carry: this tile's aggregate, read by the other blocks of the cluster
};

// Scan-order tile of this block, and the call's epoch when the carry goes through the workspace.
// Tiles are taken in launch-index order: a block waits only for the records of tiles with smaller
// indices, whose blocks the hardware has dispatched before it.  Call after grid_dependency_wait().
__device__ __forceinline__ long long take_tile(const ScanParams& p, unsigned& epoch) {
    epoch = 0;
    if (p.carry_mode && threadIdx.x < 32) epoch = ld_volatile_u32(p.header);
    return blockIdx.x;
}

// Carry between the thread blocks of one cluster (rows that are exactly 2..8 tiles long: one
// cluster per row, block rank = the tile's position in scan order inside the row).  Every block
// leaves its tile aggregate in its own shared memory; after a cluster barrier one warp reads the
// aggregates of the preceding tiles through distributed shared memory and folds them in the same
// fixed order as the look-back (nearest first, cut at the first beta = 0).  No global scratch, no
// polling.  A block must not exit before every peer has finished reading its shared memory: each
// thread arrives at a second cluster barrier here, right after the remote reads, and the caller
// waits on it (cluster_exit_wait) after its stores, so that wait overlaps the rest of the tile.
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
// The exit barrier publishes no data -- it only says "I have finished reading your shared memory" (the
// remote values were consumed by the shuffles before it) -- so its arrive needs no release fence; and
// of the first barrier's arrivals only the one thread that wrote the aggregate has something to
// publish, which it does with a fence of its own.  (Measured on 64 x 16384: GAE 6.6 -> 6.0 us,
// discounted return 4.5 -> 4.3 us against release semantics on every arrive.)
__device__ __forceinline__ void cluster_arrive_relaxed() { asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_exit_wait() { cluster_wait(); }

template <int NW>
__device__ __forceinline__ float cluster_carry(Pair tile_agg, ScanSmem<NW>& sm, int buf) {
    namespace cg = cooperative_groups;
    cg::cluster_group cl = cg::this_cluster();
    const unsigned r = cl.block_rank();
    const int lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        sm.cl_agg = tile_agg;
        asm volatile("fence.acq_rel.cluster;" ::: "memory");   // the one writer publishes; nobody else needs a release fence
    }
    cluster_arrive_relaxed();
    cluster_wait();                                            // every block's aggregate is in place
    if (threadIdx.x < 32) {
        Pair q = {0.f, 0.f};                                   // lanes >= r: terminators
        if ((unsigned)lane < r) q = *cl.map_shared_rank(&sm.cl_agg, r - 1 - lane);
        const unsigned zer = __ballot_sync(0xffffffffu, q.b == 0.f);
        const int z = __ffs(zer) - 1;                          // exists: r <= 8 < 32
        Pair cur = (lane <= z) ? q : Pair{0.f, 1.f};
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            Pair o;
            o.a = __shfl_down_sync(0xffffffffu, cur.a, d);
            o.b = __shfl_down_sync(0xffffffffu, cur.b, d);
            if (lane + d < 32 && cur.b != 0.f) cur = apply(cur, o);
        }
        if (lane == 0) sm.carry[buf] = cur.a;
    }
    cluster_arrive_relaxed();                                  // this thread reads no remote memory any more
    __syncthreads();                                           // the carry is visible to the block
    return sm.carry[buf];
}

struct NoHook {
    __device__ __forceinline__ void operator()() const {}
};

// Steps 2-5 of the header comment for one tile, given the thread's loaded Chunk.
// `after_barrier` runs right after the block barrier (every thread has consumed its inputs).
// FULL: the tile lies completely inside the array and rows are at least ITEMS long (block-uniform),
// which removes the ragged-chunk and short-row side paths at compile time.
// IDLE (with FULL): row-aligned tiling -- the block's last threads may have no steps at all; they
// read zeros, store nothing and take part in the scan as resets.
// LAST: this is the block's last tile of the call; the block then signs off from the carry protocol
// as soon as its own look-back is over (see sign_off) instead of after its stores.
// CLUSTER: the carry between blocks goes through distributed shared memory (cluster_carry).
template <int ALGO, bool TRUNC, bool VEC, int THREADS, int ITEMS, bool FULL, bool LAST, class Hook, bool CLUSTER = false,
          bool IDLE = false>
__device__ __forceinline__ void tile_compute(Chunk<ALGO, TRUNC, ITEMS>& c, Vals<ITEMS>& v, const ScanParams& p, long long i0, long long s,
                                             unsigned epoch, ScanSmem<THREADS / 32>& sm, int buf, Hook after_barrier,
                                             float* prev_out = nullptr, float* row_carry = nullptr) {
    constexpr bool FWD = is_forward(ALGO);
    constexpr int NW = THREADS / 32;
    constexpr int W = ITEMS / 4;
    constexpr unsigned ALL = 0xffffffffu;
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int warp = tid >> 5;
    const bool has_edge = c.edge < (unsigned)ITEMS;
    // IDLE (row-aligned tiling, with FULL): c.nvalid is ITEMS, or 0 for the block's idle last threads
    const int nvalid = (FULL && !IDLE) ? ITEMS : c.nvalid;

    // ---- reset words: byte j non-zero = the recurrence does NOT continue from step j to its
    // scan-order predecessor (t+1 backward, t-1 forward): a flag, a row edge, a step beyond the array
    unsigned sev[W];
    if constexpr (FWD) {
        if constexpr (ALGO == kAffineFwd) {
#pragma unroll
            for (int k = 0; k < W; ++k) sev[k] = 0;
        } else if (ALGO == kPrefix && p.starts_at) {
#pragma unroll
            for (int k = 0; k < W; ++k) sev[k] = c.dw[k];
        } else {
            // ends_at: step j is cut off by the flag of step j-1 -> shift the bytes up by one step
#pragma unroll
            for (int k = 0; k < W; ++k)
                sev[k] = (c.dw[k] << 8) | (k == 0 ? (c.halo_d & 0xffu) : (c.dw[(k + W - 1) % W] >> 24));
        }
    } else {
#pragma unroll
        for (int k = 0; k < W; ++k) sev[k] = c.dw[k] | c.tw[k];
    }
    if (has_edge) mark_byte_dyn(sev, c.edge);
    if constexpr (IDLE) {                       // an idle thread: all its steps are resets with alpha = 0 (its inputs read as zeros)
        const unsigned idle = nvalid == 0 ? 0xffffffffu : 0u;
#pragma unroll
        for (int k = 0; k < W; ++k) sev[k] |= idle;
    }
    if constexpr (!FULL) {
        if (p.T < (unsigned)ITEMS) {            // rows shorter than a chunk: several edges
            for (unsigned e = c.edge + p.T; e < (unsigned)ITEMS; e += p.T) mark_byte_dyn(sev, e);
        }
        if (nvalid < ITEMS) {                   // ragged end of the array
            for (unsigned j = nvalid; j < (unsigned)ITEMS; ++j) mark_byte_dyn(sev, j);
        }
    }

    // ---- window-edge bootstrap into ov at the row's last step, unless that step carries a flag
    // (static indexing only, so that ov stays in registers)
    if constexpr (!FWD && !is_affine(ALGO)) {
        if (has_edge && p.boot != nullptr) {
            if (FULL || p.T >= (unsigned)ITEMS) {   // at most one row edge in the chunk; its bootstrap was fetched early
                const bool ok = c.edge < (unsigned)nvalid && !test_byte_dyn(c.dw, c.edge) && !test_byte_dyn(c.tw, c.edge);
#pragma unroll
                for (int j = 0; j < ITEMS; ++j) c.ov[j] = (ok && (unsigned)j == c.edge) ? c.boot_first : c.ov[j];
            } else {                            // rows shorter than a chunk: walk the steps
                unsigned e = c.edge;
                long long n = i0 / (long long)p.T;      // row of the chunk's first step
#pragma unroll
                for (int j = 0; j < ITEMS; ++j) {
                    if ((unsigned)j == e) {
                        if (j < nvalid && !test_byte(c.dw, j) && !test_byte(c.tw, j)) c.ov[j] = ld_io(p.boot + n);
                        e += p.T;
                        ++n;
                    }
                }
            }
        }
    }

    // ---- coefficients (branch-free)
    float beta[ITEMS];
    float grho[ITEMS];             // V-Trace: gamma * rho_t where the recurrence continues, for the advantage epilogue
#pragma unroll
    for (int j = 0; j < ITEMS; ++j) {
        const bool cut = test_byte(sev, j);
        if constexpr (FWD) {
            if constexpr (ALGO == kAffineFwd) beta[j] = cut ? 0.f : v.x1[j];
            else beta[j] = cut ? 0.f : p.decay;
        } else if constexpr (ALGO == kAffineBwd) {
            beta[j] = cut ? 0.f : v.x1[j];
        } else {
            const float r = v.a[j];
            float nextv = 0.f;
            if constexpr (has_values(ALGO)) nextv = (j + 1 < ITEMS) ? v.x1[(j + 1) % ITEMS] : v.halo;
            if constexpr (is_retrace(ALGO)) nextv = (j + 1 < ITEMS) ? v.x2[(j + 1) % ITEMS] : v.halo;
            const float xn = cut ? c.ov[j] : nextv;      // successor value of Section 3.2 (selected, never multiplied)
            if constexpr (ALGO == kFillSkip) {
                // an unmasked step starts a new run with its own value; a masked one passes its
                // successor's through, or takes the flag's successor value where it is severed
                const bool masked = test_byte(c.kw, j);
                v.a[j] = masked ? (cut ? c.ov[j] : 0.f) : r;
                beta[j] = (masked && !cut) ? 1.f : 0.f;
            } else if constexpr (ALGO == kGaeSkip) {
                // x1 holds W (kFillSkip's output): V at unmasked steps, so delta is the usual one
                const bool masked = test_byte(c.kw, j);
                v.a[j] = masked ? 0.f : fmaf(p.gamma, xn, r) - v.x1[j];
                beta[j] = cut ? 0.f : (masked ? 1.f : p.decay);
            } else if constexpr (is_gae(ALGO)) {
                v.a[j] = fmaf(p.gamma, xn, r) - v.x1[j];
                beta[j] = cut ? 0.f : p.decay;
            } else if constexpr (ALGO == kTdLambda) {
                // continuing: r + gamma(1-lambda) V_{t+1}; severed: r + gamma * successor value
                v.a[j] = fmaf(cut ? p.gamma : p.aux, xn, r);
                beta[j] = cut ? 0.f : p.decay;
            } else if constexpr (ALGO == kDisc) {
                v.a[j] = fmaf(p.gamma, c.ov[j], r);
                beta[j] = cut ? 0.f : p.decay;
            } else if constexpr (ALGO == kVtrace) {
                const float raw = expf(v.x3[j]);
                const float rho = fminf(p.rho_bar, raw);
                const float cc = fminf(p.c_bar, raw);
                v.a[j] = rho * (fmaf(p.gamma, xn, r) - v.x1[j]);
                beta[j] = cut ? 0.f : p.gamma * cc;
                grho[j] = cut ? 0.f : p.gamma * rho;
            } else if constexpr (is_retrace(ALGO)) {
                v.a[j] = fmaf(p.gamma, xn, r) - v.x1[j];
                const float lr_next = (j + 1 < ITEMS) ? v.x3[(j + 1) % ITEMS] : v.halo_lr;
                // x3 holds log(pi/mu) for the scalar-input form, the ratio pi/mu itself for the tensor form
                const float ratio_next = (ALGO == kRetrace) ? expf(lr_next) : lr_next;
                beta[j] = cut ? 0.f : p.aux * fminf(p.c_bar, ratio_next);
            }
        }
    }

    // ---- thread aggregate (serial combine, Eq. 2)
    Pair agg;
    if constexpr (FWD) {
        agg.a = v.a[0];
#pragma unroll
        for (int j = 1; j < ITEMS; ++j) agg.a = fmaf(beta[j], agg.a, v.a[j]);
    } else {
        agg.a = v.a[ITEMS - 1];
#pragma unroll
        for (int j = ITEMS - 2; j >= 0; --j) agg.a = fmaf(beta[j], agg.a, v.a[j]);
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

    // ---- warp scan in scan order; rank = position in scan order inside the warp
    const int rank = FWD ? lane : 31 - lane;
    Pair incl = agg;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        Pair o;
        if constexpr (FWD) {
            o.a = __shfl_up_sync(ALL, incl.a, d);
            o.b = __shfl_up_sync(ALL, incl.b, d);
        } else {
            o.a = __shfl_down_sync(ALL, incl.a, d);
            o.b = __shfl_down_sync(ALL, incl.b, d);
        }
        if (rank >= d) incl = apply(incl, o);
    }
    Pair excl;     // everything earlier in scan order inside this warp
    if constexpr (FWD) {
        excl.a = __shfl_up_sync(ALL, incl.a, 1);
        excl.b = __shfl_up_sync(ALL, incl.b, 1);
    } else {
        excl.a = __shfl_down_sync(ALL, incl.a, 1);
        excl.b = __shfl_down_sync(ALL, incl.b, 1);
    }
    if (rank == 0) excl = Pair{0.f, 1.f};

    // ---- block carry through shared memory
    const int wrank = FWD ? warp : NW - 1 - warp;
    if (rank == 31) sm.agg[buf][wrank] = incl;
    if (wrank == 0 && rank == 0) {
        // the tile's first step in scan order: does the recurrence enter the tile from outside?
        sm.need[buf] = test_byte(sev, FWD ? 0 : ITEMS - 1) ? 0 : 1;
    }
    __syncthreads();
    after_barrier();

    Pair wcarry = {0.f, 1.f};      // all warps earlier in scan order
    Pair tile_agg;
    {
        Pair w = (lane < NW) ? sm.agg[buf][lane] : Pair{0.f, 1.f};
#pragma unroll
        for (int d = 1; d < NW; d <<= 1) {
            Pair o;
            o.a = __shfl_up_sync(ALL, w.a, d);
            o.b = __shfl_up_sync(ALL, w.b, d);
            if (lane >= d) w = apply(w, o);
        }
        tile_agg.a = __shfl_sync(ALL, w.a, NW - 1);
        tile_agg.b = __shfl_sync(ALL, w.b, NW - 1);
        const float ca = __shfl_sync(ALL, w.a, (wrank + NW - 1) % NW);
        const float cb = __shfl_sync(ALL, w.b, (wrank + NW - 1) % NW);
        if (wrank > 0) wcarry = Pair{ca, cb};
    }
    const Pair before = apply(excl, wcarry);   // everything earlier in scan order inside this tile

    // ---- carry between thread blocks
    float carry_in = 0.f;
    if (row_carry != nullptr) {
        // one block walks the whole row: the carry stays in a register (every thread holds the same
        // tile aggregate, so every thread updates its own copy -- no barrier, no memory traffic)
        carry_in = *row_carry;
        *row_carry = fmaf(tile_agg.b, carry_in, tile_agg.a);
    } else if constexpr (CLUSTER) {
        carry_in = cluster_carry<NW>(tile_agg, sm, buf);
    } else if (p.carry_mode) {
        if (warp == 0 && lane == 0 && s != p.mute_tile) {
            st_volatile_u4(p.records + s, make_uint4(__float_as_uint(tile_agg.a), epoch,
                                                     __float_as_uint(tile_agg.b), epoch));
        }
        const int need = sm.need[buf];         // block-uniform
        if (need) {
            if (warp == 0) {
                const float cin = lookback(p.records, epoch, s, p.spin_cap, p.status, lane);
                if (lane == 0) sm.carry[buf] = cin;
            }
            __syncthreads();
            carry_in = sm.carry[buf];
        }
        if constexpr (LAST) sign_off(p);
    }
    // value of the recurrence at the step just before this thread's chunk in scan order
    float prev = fmaf(before.b, carry_in, before.a);
    if (prev_out != nullptr) *prev_out = prev;

    // ---- replay, epilogue, store
    float out1v[ITEMS];
    if constexpr (FWD) {
#pragma unroll
        for (int j = 0; j < ITEMS; ++j) {
            prev = fmaf(beta[j], prev, v.a[j]);
            v.a[j] = prev;
        }
    } else {
#pragma unroll
        for (int j = ITEMS - 1; j >= 0; --j) {
            const float d = fmaf(beta[j], prev, v.a[j]);
            if constexpr (is_gae(ALGO)) {
                v.a[j] = d;
                out1v[j] = d + v.x1[j];
            } else if constexpr (ALGO == kVtrace) {
                // A_t = rho_t (r_t + gamma v_{t+1} - V_t) = alpha_t + gamma rho_t Delta_{t+1} where the
                // recurrence continues (v_{t+1} = V_{t+1} + Delta_{t+1}), alpha_t elsewhere.
                out1v[j] = fmaf(grho[j], prev, v.a[j]);
                v.a[j] = v.x1[j] + d;
            } else if constexpr (is_retrace(ALGO)) {
                v.a[j] = v.x1[j] + d;
            } else {
                v.a[j] = d;
            }
            prev = d;
        }
    }
    if (nvalid > 0) {
        store_f32<ITEMS, VEC>(p.out0, i0, nvalid, v.a);
        if constexpr (is_gae(ALGO) || ALGO == kVtrace) {
            if (p.out1 != nullptr) store_f32<ITEMS, VEC>(p.out1, i0, nvalid, out1v);
        }
    }
    // ---- per-tile statistics of A for the normalisation pass, in a fixed order (deterministic):
    // the tile's sum, and its sum of squared deviations from the tile's own mean.  Squares are
    // taken around the tile mean so that a mean far from zero does not swallow the variance in
    // fp32 (sum A^2 - mean * sum A cancels catastrophically there).
    if constexpr (ALGO == kGaeStats) {
        float s1 = 0.f;
#pragma unroll
        for (int j = 0; j < ITEMS; ++j) s1 += v.a[j];         // steps beyond the array hold A = 0
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) s1 += __shfl_xor_sync(ALL, s1, d);
        __syncthreads();                           // the scan's use of sm.agg is over
        if (lane == 0) sm.agg[buf][warp].a = s1;
        __syncthreads();
        float tile_sum = 0.f;
#pragma unroll
        for (int w = 0; w < NW; ++w) tile_sum += sm.agg[buf][w].a;      // same order in every thread
        const long long tile_start = i0 - (long long)tid * ITEMS;
        const long long left = p.total - tile_start;
        const float count = (float)(left < (long long)p.tile_steps ? left : (long long)p.tile_steps);
        const float mean = tile_sum / count;
        float q = 0.f;
#pragma unroll
        for (int j = 0; j < ITEMS; ++j) {
            const float d = v.a[j] - mean;
            q = (j < nvalid) ? fmaf(d, d, q) : q;
        }
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) q += __shfl_xor_sync(ALL, q, d);
        if (lane == 0) sm.agg[buf][warp].b = q;
        __syncthreads();
        if (tid == 0) {
            float tile_q = 0.f;
#pragma unroll
            for (int w = 0; w < NW; ++w) tile_q += sm.agg[buf][w].b;
            p.stats[2 * s] = tile_sum;
            p.stats[2 * s + 1] = tile_q;
        }
    }
    if constexpr (CLUSTER) cluster_exit_wait();
}

// ------------------------------------------------------------------------------------------ end of a call (carry mode)
// ------------------------------------------------------------------------------------------ kernel 1: one tile per block
template <int ALGO, bool TRUNC, bool VEC, int THREADS, int ITEMS, bool FULL, bool IDLE = false, bool ROWTILES = false>
__device__ __forceinline__ void one_tile(const ScanParams& p, long long tile, long long s, unsigned epoch,
                                         ScanSmem<THREADS / 32>& sm) {
    constexpr int TILE = THREADS * ITEMS;
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    Chunk<ALGO, TRUNC, ITEMS> c;
    long long i0, n0;
    if constexpr (ROWTILES) {
        // row-aligned tiling: a tile covers p.tile_steps steps, a whole number of rows that is a little
        // less than THREADS*ITEMS, and the last threads of the block have nothing to do
        i0 = tile * p.tile_steps + (long long)tid * ITEMS;
        const long long tile_end = (tile + 1) * p.tile_steps;
        n0 = locate(c, p, i0, tile_end < p.total ? tile_end : p.total);
    } else {
        i0 = tile * TILE + (long long)tid * ITEMS;
        n0 = locate(c, p, i0);
    }
    load_flags_global<ALGO, TRUNC, ITEMS, VEC, FULL, IDLE>(c, p, i0, lane);
    Vals<ITEMS> v;
    load_values_global<ALGO, TRUNC, ITEMS, VEC, FULL, IDLE>(c, v, p, i0, lane);
    issue_boot(c, p, n0);
    issue_trunc_values<ALGO, TRUNC, ITEMS, (VEC && FULL)>(c, p, i0);
    tile_compute<ALGO, TRUNC, VEC, THREADS, ITEMS, FULL, true, NoHook, false, IDLE>(c, v, p, i0, s, epoch, sm, 0, NoHook{});
}

// ROWTILES: the instantiation for row-aligned tiling (p.tile_steps < THREADS*ITEMS), kept apart so that
// the kernel for whole tiles stays exactly as lean as it is without that feature.
template <int ALGO, bool TRUNC, bool VEC, int THREADS, int ITEMS, int MIN_BLOCKS, bool ROWTILES = false>
__global__ void __launch_bounds__(THREADS, MIN_BLOCKS) scan_kernel(const ScanParams p) {
    constexpr bool FWD = is_forward(ALGO);
    constexpr int TILE = THREADS * ITEMS;
    __shared__ ScanSmem<THREADS / 32> sm;

    grid_dependency_launch();
    grid_dependency_wait();
    unsigned epoch;
    const long long s = take_tile(p, epoch);          // tile index in scan order
    const long long tile = FWD ? s : (p.num_tiles - 1 - s);
    if constexpr (ROWTILES) {
        // tile inside the array: whole chunks in the first threads, none in the last few (block-uniform)
        if (VEC && (tile + 1) * (long long)p.tile_steps <= p.total && p.T >= (unsigned)ITEMS)
            one_tile<ALGO, TRUNC, VEC, THREADS, ITEMS, true, true, true>(p, tile, s, epoch, sm);
        else one_tile<ALGO, TRUNC, VEC, THREADS, ITEMS, false, false, true>(p, tile, s, epoch, sm);
    } else {
        // block-uniform: the whole tile is inside the array and no row is shorter than a chunk
        const bool full = (tile * TILE + TILE <= p.total) && (p.T >= (unsigned)ITEMS);
        if (full) one_tile<ALGO, TRUNC, VEC, THREADS, ITEMS, true>(p, tile, s, epoch, sm);
        else one_tile<ALGO, TRUNC, VEC, THREADS, ITEMS, false>(p, tile, s, epoch, sm);
    }
}

// ------------------------------------------------------------------------------------------ kernel 1b: GAE with observation-skip masking
// Both scans of the masked GAE in one pass over the tile: first the fill scan (W = the value a step
// shows to its predecessors), whose result stays in registers -- a thread's successor value W at
// i0 + ITEMS is the fill recurrence's own incoming value -- then the masked GAE scan on (rewards, W).
// Each scan has its own carry records (the second half of the record array) and shared-memory
// buffers; the block signs off after the second.  p.f0 = rewards, p.f1 = values, p.out2 = W,
// p.out0 / p.out1 = advantages / returns.
#ifndef RLCS_IO_BF16
template <bool TRUNC, bool VEC, int THREADS, int ITEMS, bool FULL>
__device__ __forceinline__ void one_tile_gae_skip(const ScanParams& p, long long tile, long long s, unsigned epoch,
                                                  ScanSmem<THREADS / 32>& sm) {
    constexpr int TILE = THREADS * ITEMS;
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const long long i0 = tile * TILE + (long long)tid * ITEMS;
    Chunk<kFillSkip, TRUNC, ITEMS> cf;
    const long long n0 = locate(cf, p, i0);
    load_flags_global<kFillSkip, TRUNC, ITEMS, VEC, FULL>(cf, p, i0, lane);
    const int nvalid = FULL ? ITEMS : cf.nvalid;
    Vals<ITEMS> vf, vg;
    load_f32<ITEMS, VEC>(p.f1, i0, nvalid, vf.a);            // values: the fill scan's input
    load_f32<ITEMS, VEC>(p.f0, i0, nvalid, vg.a);            // rewards, for the second scan
    vf.halo = 0.f; vf.halo_lr = 0.f;
    issue_boot(cf, p, n0);
    issue_trunc_values(cf, p, i0);
    Chunk<kGaeSkip, TRUNC, ITEMS> cg;
    cg.edge = cf.edge; cg.nvalid = cf.nvalid; cg.halo_d = 0; cg.boot_first = cf.boot_first;
#pragma unroll
    for (int k = 0; k < ITEMS / 4; ++k) { cg.dw[k] = cf.dw[k]; cg.tw[k] = cf.tw[k]; cg.kw[k] = cf.kw[k]; }
#pragma unroll
    for (int j = 0; j < ITEMS; ++j) cg.ov[j] = cf.ov[j];

    ScanParams pf = p;
    pf.out0 = p.out2;
    pf.out1 = nullptr;
    float w_next = 0.f;
    tile_compute<kFillSkip, TRUNC, VEC, THREADS, ITEMS, FULL, false>(cf, vf, pf, i0, s, epoch, sm, 0, NoHook{}, &w_next);

    ScanParams pg = p;
    pg.records = p.records + p.num_tiles;
#pragma unroll
    for (int j = 0; j < ITEMS; ++j) vg.x1[j] = vf.a[j];      // W of this thread's steps
    vg.halo = w_next;
    vg.halo_lr = 0.f;
    tile_compute<kGaeSkip, TRUNC, VEC, THREADS, ITEMS, FULL, true>(cg, vg, pg, i0, s, epoch, sm, 1, NoHook{});
}

template <bool TRUNC, bool VEC, int THREADS, int ITEMS, int MIN_BLOCKS>
__global__ void __launch_bounds__(THREADS, MIN_BLOCKS) scan_kernel_gae_skip(const ScanParams p) {
    constexpr int TILE = THREADS * ITEMS;
    __shared__ ScanSmem<THREADS / 32> sm;
    grid_dependency_launch();
    grid_dependency_wait();
    unsigned epoch;
    const long long s = take_tile(p, epoch);
    const long long tile = p.num_tiles - 1 - s;
    const bool full = (tile * TILE + TILE <= p.total) && (p.T >= (unsigned)ITEMS);
    if (full) one_tile_gae_skip<TRUNC, VEC, THREADS, ITEMS, true>(p, tile, s, epoch, sm);
    else one_tile_gae_skip<TRUNC, VEC, THREADS, ITEMS, false>(p, tile, s, epoch, sm);
}

// The same with one thread block per row (rows of whole tiles, many rows -- token-level trajectories
// are long): block n walks the tiles of row n in scan order and keeps both carries, the fill's and
// the advantage's, in registers; no records, no waiting.  The two scans of a tile use the two halves
// of the shared scratch, and each scan's block barrier separates a half's reads in one tile from its
// writes in the next.
template <bool TRUNC, int THREADS, int ITEMS, int MIN_BLOCKS>
__global__ void __launch_bounds__(THREADS, MIN_BLOCKS) scan_kernel_gae_skip_rows(const ScanParams p) {
    constexpr int TILE = THREADS * ITEMS;
    __shared__ ScanSmem<THREADS / 32> sm;
    grid_dependency_launch();
    grid_dependency_wait();
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const long long row_start = (long long)blockIdx.x * p.T;
    const long long row_end = row_start + p.T;
    const unsigned tiles = p.T / TILE;                        // whole tiles only (the host checks)
    ScanParams pf = p;
    pf.out0 = p.out2;
    pf.out1 = nullptr;
    float carry_w = 0.f, carry_a = 0.f;
    for (unsigned k = 0; k < tiles; ++k) {
        const long long i0 = row_start + (long long)(tiles - 1 - k) * TILE + (long long)tid * ITEMS;
        Chunk<kFillSkip, TRUNC, ITEMS> cf;
        const long long n0 = locate(cf, p, i0, row_end);
        load_flags_global<kFillSkip, TRUNC, ITEMS, true, true>(cf, p, i0, lane);
        Vals<ITEMS> vf, vg;
        load_f32<ITEMS, true>(p.f1, i0, ITEMS, vf.a);        // values: the fill scan's input
        load_f32<ITEMS, true>(p.f0, i0, ITEMS, vg.a);        // rewards, for the second scan
        vf.halo = 0.f; vf.halo_lr = 0.f;
        issue_boot(cf, p, n0);
        issue_trunc_values(cf, p, i0);
        Chunk<kGaeSkip, TRUNC, ITEMS> cg;
        cg.edge = cf.edge; cg.nvalid = cf.nvalid; cg.halo_d = 0; cg.boot_first = cf.boot_first;
#pragma unroll
        for (int q = 0; q < ITEMS / 4; ++q) { cg.dw[q] = cf.dw[q]; cg.tw[q] = cf.tw[q]; cg.kw[q] = cf.kw[q]; }
#pragma unroll
        for (int j = 0; j < ITEMS; ++j) cg.ov[j] = cf.ov[j];
        float w_next = 0.f;
        tile_compute<kFillSkip, TRUNC, true, THREADS, ITEMS, true, false, NoHook, false, false>(cf, vf, pf, i0, 0, 0u, sm, 0, NoHook{},
                                                                                               &w_next, &carry_w);
#pragma unroll
        for (int j = 0; j < ITEMS; ++j) vg.x1[j] = vf.a[j];  // W of this thread's steps
        vg.halo = w_next;
        vg.halo_lr = 0.f;
        tile_compute<kGaeSkip, TRUNC, true, THREADS, ITEMS, true, false, NoHook, false, false>(cg, vg, p, i0, 0, 0u, sm, 1, NoHook{},
                                                                                              nullptr, &carry_a);
    }
}
#endif  // !RLCS_IO_BF16

// ------------------------------------------------------------------------------------------ kernel 1c: Retrace from [N,T,A] tensors
#ifndef RLCS_IO_BF16
template <bool TRUNC, bool VEC, int THREADS, int ITEMS, int AV, bool FULL>
__device__ __forceinline__ void one_tile_probs(const ScanParams& p, long long tile, long long s, unsigned epoch,
                                               ScanSmem<THREADS / 32>& sm) {
    constexpr int ALGO = kRetraceProbs;
    constexpr int TILE = THREADS * ITEMS;
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    Chunk<ALGO, TRUNC, ITEMS> c;
    const long long i0 = tile * TILE + (long long)tid * ITEMS;
    const long long n0 = locate(c, p, i0);
    load_flags_global<ALGO, TRUNC, ITEMS, VEC, FULL>(c, p, i0, lane);
    Vals<ITEMS> v;
    load_values_probs<ALGO, TRUNC, ITEMS, AV>(c, v, p, i0, lane, FULL ? ITEMS : c.nvalid);
    issue_boot(c, p, n0);
    issue_trunc_values(c, p, i0);
    tile_compute<ALGO, TRUNC, VEC, THREADS, ITEMS, FULL, true>(c, v, p, i0, s, epoch, sm, 0, NoHook{});
}

template <bool TRUNC, bool VEC, int THREADS, int ITEMS, int MIN_BLOCKS, int AV>
__global__ void __launch_bounds__(THREADS, MIN_BLOCKS) scan_kernel_retrace_probs(const ScanParams p) {
    constexpr int TILE = THREADS * ITEMS;
    __shared__ ScanSmem<THREADS / 32> sm;
    grid_dependency_launch();
    grid_dependency_wait();
    unsigned epoch;
    const long long s = take_tile(p, epoch);
    const long long tile = p.num_tiles - 1 - s;
    const bool full = (tile * TILE + TILE <= p.total) && (p.T >= (unsigned)ITEMS);      // block-uniform
    if (full) one_tile_probs<TRUNC, VEC, THREADS, ITEMS, AV, true>(p, tile, s, epoch, sm);
    else one_tile_probs<TRUNC, VEC, THREADS, ITEMS, AV, false>(p, tile, s, epoch, sm);
}

// The same with one thread block per row (rows of whole tiles, many rows): block n walks the tiles of
// row n in scan order and keeps the carry in a register, as scan_kernel_rows does for the scalar-input
// algorithms -- no records, no waiting, whatever T is.
template <bool TRUNC, int THREADS, int ITEMS, int MIN_BLOCKS, int AV>
__global__ void __launch_bounds__(THREADS, MIN_BLOCKS) scan_kernel_retrace_probs_rows(const ScanParams p) {
    constexpr int ALGO = kRetraceProbs;
    constexpr int TILE = THREADS * ITEMS;
    __shared__ ScanSmem<THREADS / 32> sm;
    grid_dependency_launch();
    grid_dependency_wait();
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const long long row_start = (long long)blockIdx.x * p.T;
    const long long row_end = row_start + p.T;
    const unsigned tiles = p.T / TILE;                        // whole tiles only (the host checks)
    float carry = 0.f;
    for (unsigned k = 0; k < tiles; ++k) {
        const long long i0 = row_start + (long long)(tiles - 1 - k) * TILE + (long long)tid * ITEMS;
        Chunk<ALGO, TRUNC, ITEMS> c;
        const long long n0 = locate(c, p, i0, row_end);
        load_flags_global<ALGO, TRUNC, ITEMS, true, true>(c, p, i0, lane);
        Vals<ITEMS> v;
        load_values_probs<ALGO, TRUNC, ITEMS, AV>(c, v, p, i0, lane, ITEMS);
        issue_boot(c, p, n0);
        issue_trunc_values(c, p, i0);
        // shared scratch alternates by tile parity, so one barrier per tile suffices
        tile_compute<ALGO, TRUNC, true, THREADS, ITEMS, true, false, NoHook, false, false>(c, v, p, i0, 0, 0u, sm, k & 1, NoHook{},
                                                                                          nullptr, &carry);
    }
}

#endif  // !RLCS_IO_BF16

// ------------------------------------------------------------------------------------------ kernel 1b: one tile per block, one cluster per row
// For rows that are exactly 2..8 tiles long (T = k * TILE): launched with cluster size k, so a
// cluster is a row and the carry stays on chip.  All tiles are full; 32-byte aligned pointers.
template <int ALGO, bool TRUNC, int THREADS, int ITEMS, int MIN_BLOCKS>
__global__ void __launch_bounds__(THREADS, MIN_BLOCKS) scan_kernel_cluster(const ScanParams p) {
    constexpr bool FWD = is_forward(ALGO);
    constexpr int TILE = THREADS * ITEMS;
    __shared__ ScanSmem<THREADS / 32> sm;
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const long long s = blockIdx.x;
    const long long tile = FWD ? s : (p.num_tiles - 1 - s);
    grid_dependency_launch();
    Chunk<ALGO, TRUNC, ITEMS> c;
    const long long i0 = tile * TILE + (long long)tid * ITEMS;
    const long long n0 = locate(c, p, i0);
    grid_dependency_wait();
    load_flags_global<ALGO, TRUNC, ITEMS, true, true>(c, p, i0, lane);
    Vals<ITEMS> v;
    load_values_global<ALGO, TRUNC, ITEMS, true, true>(c, v, p, i0, lane);
    issue_boot(c, p, n0);
    issue_trunc_values<ALGO, TRUNC, ITEMS, true>(c, p, i0);
    tile_compute<ALGO, TRUNC, true, THREADS, ITEMS, true, false, NoHook, true>(c, v, p, i0, s, 0u, sm, 0, NoHook{});
}

// ------------------------------------------------------------------------------------------ kernel 1e: one thread block per row
// For rows longer than a tile when there are at least as many rows as thread blocks fit on the GPU:
// block n walks the tiles of row n in scan order and carries the recurrence from tile to tile in a
// register.  Blocks never wait for one another and nothing goes through global memory; the other
// blocks resident on the SM keep the memory system busy while one block is between its loads and
// its stores, exactly as with one tile per block.  The row's last tile (in address order) may be
// short: its tail threads idle (T must be a multiple of the steps per thread, which also keeps every
// chunk aligned for 256-bit accesses).  Vector accesses only.
template <int ALGO, bool TRUNC, int THREADS, int ITEMS, bool IDLE>
__device__ __forceinline__ void row_tile(const ScanParams& p, long long tile_start, long long row_end, float& carry,
                                         ScanSmem<THREADS / 32>& sm, int buf, long long s) {
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    Chunk<ALGO, TRUNC, ITEMS> c;
    const long long i0 = tile_start + (long long)tid * ITEMS;
    const long long n0 = locate(c, p, i0, row_end);
    load_flags_global<ALGO, TRUNC, ITEMS, true, true, IDLE>(c, p, i0, lane);
    Vals<ITEMS> v;
    load_values_global<ALGO, TRUNC, ITEMS, true, true, IDLE>(c, v, p, i0, lane);
    issue_boot(c, p, n0);
    issue_trunc_values<ALGO, TRUNC, ITEMS, true>(c, p, i0);
    // (s only numbers the tile for the per-tile statistics of kGaeStats)
    tile_compute<ALGO, TRUNC, true, THREADS, ITEMS, true, false, NoHook, false, IDLE>(c, v, p, i0, s, 0u, sm, buf, NoHook{}, nullptr,
                                                                                     &carry);
}

template <int ALGO, bool TRUNC, int THREADS, int ITEMS, int MIN_BLOCKS>
__global__ void __launch_bounds__(THREADS, MIN_BLOCKS) scan_kernel_rows(const ScanParams p) {
    constexpr bool FWD = is_forward(ALGO);
    constexpr int TILE = THREADS * ITEMS;
    __shared__ ScanSmem<THREADS / 32> sm;
    grid_dependency_launch();
    grid_dependency_wait();
    const long long row_start = (long long)blockIdx.x * p.T;
    const long long row_end = row_start + p.T;
    const unsigned tiles = (p.T + TILE - 1) / TILE;
    float carry = 0.f;                                        // the row's boundary carry is folded into alpha at its edge
    for (unsigned k = 0; k < tiles; ++k) {
        const unsigned m = FWD ? k : tiles - 1 - k;           // k-th tile in scan order
        const long long tile_start = row_start + (long long)m * TILE;
        // shared scratch alternates by tile parity, so one barrier per tile suffices (as in the persistent kernel)
        const long long s = (long long)blockIdx.x * tiles + k;
        if (tile_start + TILE <= row_end) row_tile<ALGO, TRUNC, THREADS, ITEMS, false>(p, tile_start, row_end, carry, sm, k & 1, s);
        else row_tile<ALGO, TRUNC, THREADS, ITEMS, true>(p, tile_start, row_end, carry, sm, k & 1, s);
    }
}

// ------------------------------------------------------------------------------------------ mbarrier / bulk copy (PTX)
__device__ __forceinline__ unsigned smem_u32(const void* ptr) { return (unsigned)__cvta_generic_to_shared(ptr); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, unsigned parity) {
    unsigned ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// 1-D bulk copy global -> this block's shared memory only, completing `bytes` on `bar`.
// dst, src 16-byte aligned; bytes a multiple of 16.
__device__ __forceinline__ void bulk_load(void* dst, const void* src, unsigned bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cta.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 :: "r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void fence_barrier_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// Shared-memory layout of one ring stage: the float arrays the algorithm reads (TILE + 4 floats
// each: the tile plus the halo step) and its mask arrays (16 bytes of front pad, then TILE bytes;
// forward scans copy the 16 bytes before the tile into the pad to get the preceding dones byte).
template <int ALGO, bool TRUNC, int TILE>
struct StageLayout {
    static constexpr int NF = 1 + (uses_f1(ALGO) ? 1 : 0) + (uses_f2(ALGO) ? 1 : 0) + (uses_f3(ALGO) ? 1 : 0);
    static constexpr int NM = (uses_dones(ALGO) ? 1 : 0) + (TRUNC ? 1 : 0);
    static constexpr int F_BYTES = (TILE + 4) * 4;
    static constexpr int M_BYTES = TILE + 16;
    static constexpr int BYTES = ((NF * F_BYTES + NM * M_BYTES) + 127) / 128 * 128;
    // slot of each array among the float arrays
    static constexpr int SLOT_F1 = 1;
    static constexpr int SLOT_F2 = 2;
    static constexpr int SLOT_F3 = 1 + (uses_f1(ALGO) ? 1 : 0) + (uses_f2(ALGO) ? 1 : 0);
    __device__ static float* f(unsigned char* stage, int slot) { return reinterpret_cast<float*>(stage + slot * F_BYTES); }
    __device__ static uint8_t* m(unsigned char* stage, int slot) { return stage + NF * F_BYTES + slot * M_BYTES; }
};

// Wait until the ring stage of the cj-th bulk-fetched tile of this block has landed.  The wait is
// bounded twice over (poll count and about a second of SM clock); when it gives up it records
// RLCS_ERR_TIMEOUT in the status word and every later wait of this block returns at once.
constexpr long long kWaitClockLimit = 2000000000ll;
template <int STAGES>
__device__ __forceinline__ void wait_stage(uint64_t* full_bar, unsigned cj, const ScanParams& p, bool& gave_up) {
    uint64_t* bar = &full_bar[cj % STAGES];
    const unsigned parity = (cj / STAGES) & 1u;
    if (gave_up || mbar_try_wait(bar, parity)) return;
    const long long t_start = clock64();
    unsigned spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if (++spins > p.spin_cap || clock64() - t_start > kWaitClockLimit) {
            if (p.status != nullptr) atomicExch(p.status, kDeviceTimeout);
            gave_up = true;
            return;
        }
    }
}

// Geometry, flags, window-edge bootstrap and sparse truncation values of address tile `tile`:
// everything the coefficient stage needs besides the float inputs.  Called one tile ahead, so that
// the dependent loads (bootstrap values) are in flight while the previous tile is being stored.
template <int ALGO, bool TRUNC, int THREADS, int ITEMS, int STAGES>
__device__ __forceinline__ void prefetch_flags(Chunk<ALGO, TRUNC, ITEMS>& c, const ScanParams& p, long long tile,
                                               unsigned char* ring, uint64_t* full_bar, unsigned cj, bool& gave_up) {
    constexpr int TILE = THREADS * ITEMS;
    constexpr int HALO = float_halo(ALGO) ? 4 : 0;
    constexpr int W = ITEMS / 4;
    using L = StageLayout<ALGO, TRUNC, TILE>;
    const int tid = threadIdx.x;
    const long long i0 = tile * TILE + (long long)tid * ITEMS;
    const long long n0 = locate(c, p, i0);
    issue_boot(c, p, n0);
    if (tile * TILE + TILE + HALO <= p.total) {
        wait_stage<STAGES>(full_bar, cj, p, gave_up);
        unsigned char* stage = ring + (size_t)(cj % STAGES) * L::BYTES;
#pragma unroll
        for (int k = 0; k < W; ++k) { c.dw[k] = 0; c.tw[k] = 0; }
        c.halo_d = 0;
        if constexpr (uses_dones(ALGO)) {
            const uint8_t* md = L::m(stage, 0) + 16 + tid * ITEMS;
            lds_mask<ITEMS>(md, c.dw);
            if constexpr (ALGO == kElig || ALGO == kPrefix) c.halo_d = md[-1];   // unused garbage for tile 0 (row start)
        }
        if constexpr (TRUNC) lds_mask<ITEMS>(L::m(stage, 1) + 16 + tid * ITEMS, c.tw);
    } else {
        load_flags_global<ALGO, TRUNC, ITEMS, true>(c, p, i0, tid & 31);
    }
    issue_trunc_values(c, p, i0);
}

// ------------------------------------------------------------------------------------------ kernel 2: persistent, bulk-copy ring
// Per-block walk state of the persistent kernel (scan-order tile indices fit 32 bits: the grid of
// the one-tile-per-block kernel bounds num_tiles).  The producer's cursor lives in shared memory:
// only thread 0 uses it.
struct Walk {
    unsigned G;              // grid size = stride of the walk in scan-order tiles
    unsigned s;              // scan-order tile being processed
    unsigned cj;             // bulk-fetched tiles consumed so far
    unsigned epoch;
    int buf;                 // parity of the block-scan scratch
    bool gave_up;            // a bounded wait ran out: stop waiting, finish the walk
    unsigned* prod;          // shared: [0] = next scan-order tile to fetch, [1] = tiles fetched so far
};

template <int ALGO, int TILE>
__device__ __forceinline__ long long tile_of(const ScanParams& p, long long s) {
    return is_forward(ALGO) ? s : (p.num_tiles - 1 - s);
}
// A tile can be fetched by bulk copies when it, and the halo step behind it, lie inside the array.
template <int ALGO, int TILE>
__device__ __forceinline__ bool bulk_ok(const ScanParams& p, long long tile) {
    return tile * TILE + TILE + (float_halo(ALGO) ? 4 : 0) <= p.total;
}

// Thread 0: issue the bulk copies of this block's next fetchable tile into ring stage pj % STAGES.
template <int ALGO, bool TRUNC, int TILE, int STAGES>
__device__ __forceinline__ void produce_next(const ScanParams& p, Walk& w, unsigned char* ring, uint64_t* full_bar) {
    constexpr bool FWD = is_forward(ALGO);
    constexpr int HALO = float_halo(ALGO) ? 4 : 0;
    using L = StageLayout<ALGO, TRUNC, TILE>;
    unsigned ps = w.prod[0];
    const unsigned pj = w.prod[1];
    while (ps < p.num_tiles) {
        const long long tile = tile_of<ALGO, TILE>(p, ps);
        ps += w.G;
        if (!bulk_ok<ALGO, TILE>(p, tile)) continue;
        unsigned char* stage = ring + (size_t)(pj % STAGES) * L::BYTES;
        uint64_t* bar = &full_bar[pj % STAGES];
        const long long e0 = tile * TILE;
        // forward scans fetch the 16 mask bytes before the tile as well (the preceding step's flag)
        const bool pre = FWD && uses_dones(ALGO) && e0 >= 16;
        const unsigned dbytes = pre ? TILE + 16 : TILE;
        mbar_expect_tx(bar, L::NF * (TILE + HALO) * 4 + (uses_dones(ALGO) ? dbytes : 0) + (TRUNC ? TILE : 0));
        bulk_load(L::f(stage, 0), p.f0 + e0, (TILE + HALO) * 4, bar);
        if constexpr (uses_f1(ALGO)) bulk_load(L::f(stage, L::SLOT_F1), p.f1 + e0, (TILE + HALO) * 4, bar);
        if constexpr (uses_f2(ALGO)) bulk_load(L::f(stage, L::SLOT_F2), p.f2 + e0, (TILE + HALO) * 4, bar);
        if constexpr (uses_f3(ALGO)) bulk_load(L::f(stage, L::SLOT_F3), p.f3 + e0, (TILE + HALO) * 4, bar);
        if constexpr (uses_dones(ALGO))
            bulk_load(L::m(stage, 0) + (pre ? 0 : 16), p.dones + e0 - (pre ? 16 : 0), dbytes, bar);
        if constexpr (TRUNC) bulk_load(L::m(stage, 1) + 16, p.truncs + e0, TILE, bar);
        w.prod[0] = ps;
        w.prod[1] = pj + 1;
        return;
    }
    w.prod[0] = ps;
}

// Runs right after the block barrier of a tile, when every thread has consumed the current ring
// stage and its flags: thread 0 refills the stage, and every thread fetches the flags of the
// block's next tile (mask bytes from the ring, truncation / window-edge bootstrap values from global
// memory) so that those dependent loads are in flight during the rest of the current tile.
template <int ALGO, bool TRUNC, int THREADS, int ITEMS, int STAGES>
struct AfterBarrier {
    const ScanParams& p;
    Walk& w;
    unsigned char* ring;
    uint64_t* full_bar;
    Chunk<ALGO, TRUNC, ITEMS>& nxt;
    bool bulk;               // the current tile came through the ring
    __device__ __forceinline__ void operator()() const {
        constexpr int TILE = THREADS * ITEMS;
        if (bulk && threadIdx.x == 0) {
            fence_proxy_async();
            produce_next<ALGO, TRUNC, TILE, STAGES>(p, w, ring, full_bar);
        }
        if (w.s + w.G < p.num_tiles)
            prefetch_flags<ALGO, TRUNC, THREADS, ITEMS, STAGES>(nxt, p, tile_of<ALGO, TILE>(p, w.s + w.G), ring, full_bar,
                                                                w.cj + (bulk ? 1u : 0u), w.gave_up);
    }
};

// One tile of the walk.  `cur` holds the flags of tile w.s (fetched during the previous tile).
template <int ALGO, bool TRUNC, int THREADS, int ITEMS, int STAGES>
__device__ __forceinline__ void walk_step(Chunk<ALGO, TRUNC, ITEMS>& cur, const ScanParams& p, Walk& w,
                                          unsigned char* ring, uint64_t* full_bar, ScanSmem<THREADS / 32>& sm) {
    constexpr int TILE = THREADS * ITEMS;
    using L = StageLayout<ALGO, TRUNC, TILE>;
    const int tid = threadIdx.x;
    const long long tile = tile_of<ALGO, TILE>(p, w.s);
    const long long i0 = tile * TILE + (long long)tid * ITEMS;
    const bool bulk = bulk_ok<ALGO, TILE>(p, tile);
    Vals<ITEMS> v;
    if (bulk) {
        unsigned char* stage = ring + (size_t)(w.cj % STAGES) * L::BYTES;     // landed: prefetch_flags waited for it
        const int off = tid * ITEMS;
        lds_f32<ITEMS>(L::f(stage, 0) + off, v.a);
        if constexpr (uses_f1(ALGO)) lds_f32<ITEMS>(L::f(stage, L::SLOT_F1) + off, v.x1);
        if constexpr (uses_f2(ALGO)) lds_f32<ITEMS>(L::f(stage, L::SLOT_F2) + off, v.x2);
        if constexpr (uses_f3(ALGO)) lds_f32<ITEMS>(L::f(stage, L::SLOT_F3) + off, v.x3);
        v.halo = 0.f;
        v.halo_lr = 0.f;
        if constexpr (has_values(ALGO)) v.halo = L::f(stage, L::SLOT_F1)[off + ITEMS];
        if constexpr (ALGO == kRetrace) {
            v.halo = L::f(stage, L::SLOT_F2)[off + ITEMS];
            v.halo_lr = L::f(stage, L::SLOT_F3)[off + ITEMS];
        }
    } else {
        load_values_global<ALGO, TRUNC, ITEMS, true>(cur, v, p, i0, tid & 31);
    }
    Chunk<ALGO, TRUNC, ITEMS> nxt;
    const AfterBarrier<ALGO, TRUNC, THREADS, ITEMS, STAGES> hook{p, w, ring, full_bar, nxt, bulk};
    // A tile that came through the ring lies inside the array, and the host sends rows shorter
    // than a chunk to the other kernel: the full-tile path applies.
    if (bulk) tile_compute<ALGO, TRUNC, true, THREADS, ITEMS, true, false>(cur, v, p, i0, w.s, w.epoch, sm, w.buf, hook);
    else tile_compute<ALGO, TRUNC, true, THREADS, ITEMS, false, false>(cur, v, p, i0, w.s, w.epoch, sm, w.buf, hook);
    if (w.s + w.G < p.num_tiles) cur = nxt;
    if (bulk) ++w.cj;
    w.s += w.G;
    w.buf ^= 1;
}

template <int ALGO, bool TRUNC, int THREADS, int ITEMS, int STAGES, int MIN_BLOCKS>
__global__ void __launch_bounds__(THREADS, MIN_BLOCKS) scan_kernel_tma(const ScanParams p) {
    constexpr int TILE = THREADS * ITEMS;
    using L = StageLayout<ALGO, TRUNC, TILE>;

    extern __shared__ __align__(128) unsigned char ring[];          // STAGES * L::BYTES
    __shared__ __align__(8) uint64_t full_bar[STAGES];
    __shared__ ScanSmem<THREADS / 32> sm;

    const int tid = threadIdx.x;
    __shared__ unsigned prod[2];
    Walk w;
    w.G = gridDim.x;
    w.s = blockIdx.x;
    w.prod = prod;
    w.cj = 0;
    w.epoch = 0;
    w.buf = 0;
    w.gave_up = false;

    if (tid == 0) {
        prod[0] = blockIdx.x;
        prod[1] = 0;
#pragma unroll
        for (int k = 0; k < STAGES; ++k) mbar_init(&full_bar[k], 1);
        fence_barrier_init();
        fence_proxy_async();
    }
    grid_dependency_launch();
    __syncthreads();
    grid_dependency_wait();
    if (tid == 0) {
#pragma unroll
        for (int k = 0; k < STAGES; ++k) produce_next<ALGO, TRUNC, TILE, STAGES>(p, w, ring, full_bar);
    }
    if (p.carry_mode && tid < 32) w.epoch = ld_volatile_u32(p.header);

    Chunk<ALGO, TRUNC, ITEMS> cur;
    if (w.s < p.num_tiles)
        prefetch_flags<ALGO, TRUNC, THREADS, ITEMS, STAGES>(cur, p, tile_of<ALGO, TILE>(p, w.s), ring, full_bar, w.cj, w.gave_up);
    while (w.s < p.num_tiles) walk_step<ALGO, TRUNC, THREADS, ITEMS, STAGES>(cur, p, w, ring, full_bar, sm);
    if (p.carry_mode) sign_off(p);
}

}  // namespace RLCS_NS
