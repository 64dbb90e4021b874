// Time-major entry points: every [T, N] tensor has element (t, n) at t*N + n, the layout rollout
// buffers usually have (step-major storage of N parallel environments).
//
// The recurrence runs along t, the strided axis here, so the mapping is the transpose of the
// flat-tile kernels: a lane owns one environment n and walks its timesteps in scan order, carrying
// A_{t+1} (or A_{t-1}), the neighbouring value V(s_{t+1}) and, for Retrace, the next step's log-ratio
// in registers; the 32 lanes of a warp are 32 adjacent environments, so every row of a warp is one
// fully used 128-byte line.  The per-step arithmetic is the definition of Section 3.2 / 3.3 itself
// (successor value selected by flag, the recurrence continued only where no flag is set): no scan,
// no shuffles.
//
// Kernels that share that arithmetic:
//   * tm_block_kernel: a thread block owns 32 (or 64) adjacent environments and streams their rows
//     through a ring of shared-memory stages filled by 16-byte asynchronous copies (cp.async); its
//     warps split every stage in time (per-warp walk from carry 0, aggregates through shared memory,
//     fold, one FMA per step).  Load addresses do not depend on the recurrence, so S-1 stages are in
//     flight per block whatever the register budget.  Needs N % 16 == 0 and 16-byte aligned inputs.
//   * tm_kernel: a lane per environment walking from two alternating register blocks; any N and any
//     4-byte alignment.
//   * tm_block_chained_kernel: the block kernel over a cut time axis, in one launch (below).
//
// Parallelism is N/32 thread blocks.  When that cannot fill the GPU the time axis is cut into
// chunks.  Ring path: one launch; blocks take (column block, chunk) pairs in scan order from a
// ticket counter, walk their chunk for its aggregate (a, b) of Eq. 2, publish it, look back over
// the records of the chunks before for the carry into their own, and walk the chunk again -- out of
// L2 -- to write the outputs (the vector traces, whose flags hold for all columns at once, walk it
// only once and finish the steps before the chunk's first cut from the ring).  Register path: three
// launches (aggregates with carry 0, a small
// kernel that chains an environment's chunks in scan order, second walk from the carry), the inputs
// read twice.  Deterministic either way.
#include <cmath>
#include <cstdint>
#include <type_traits>

#include "../../include/rlcs.h"
#include "rlcs_device.cuh"
#include "rlcs_scan.cuh"

// test hooks shared with the row-major entry points (rlcs_debug_set_carry_fault; defined in rlcs_api.cu)
namespace rlcs_hooks {
extern long long g_mute_tile;      // scan-order tile / block ticket that does not publish
extern long long g_spin_cap;       // poll limit (0 = default)
extern bool g_pdl;                 // launch with programmatic stream serialisation (default on)
}  // namespace rlcs_hooks

namespace {

using rlcs::kGae;
using rlcs::kTdLambda;
using rlcs::kDisc;
using rlcs::kVtrace;
using rlcs::kRetrace;
using rlcs::kElig;
using rlcs::kPrefix;

constexpr int kRows = 8;         // timesteps per register block of tm_kernel
constexpr int kThreads = 128;    // register-path block; the staged path uses 32 * warps_per_block

struct TmParams {
    const float* f0;          // rewards | x
    const float* f1;          // values | q_sa
    const float* f2;          // expected_q
    const float* f3;          // log_rhos
    const uint8_t* dones;
    const uint8_t* truncs;
    const float* trunc_boot;  // [T,N]
    const float* boot;        // [N] or nullptr
    float* out0;
    float* out1;
    long long N;
    unsigned T;
    unsigned chunk, chunks;   // timesteps per chunk, chunks per environment (1 = time axis not cut)
    float gamma, decay, aux, rho_bar, c_bar;
    int starts_at;
    int stages, warps_per_block, cols_per_lane;   // tm_block_kernel: ring depth, warps per block, columns per lane
    long long batch, batch_stride;                // kTmVec*: independent [T, N] problems (blockIdx.z), elements between them
    float* agg_a;             // [chunks, N] pass 1: chunk aggregates; after the chain: carry into each chunk
    float* agg_b;             // [chunks, N]
    // tm_block_chained_kernel: header[63] = block ticket counter, header[2] = status word (both in the
    // workspace's first 256 bytes), records[(z * chunks + scan-order chunk) * npad + column]
    unsigned* header;
    uint4* records;
    unsigned colblocks;       // thread blocks across the columns
    long long npad;           // colblocks * 32 * cols_per_lane
    unsigned spin_cap;        // polls of one record before the kernel gives up
    long long mute_ticket;    // test hook: the block with this ticket publishes nothing (-1: none)
};

// Vector-valued eligibility traces x[n] : [T, D] are time-major problems with D columns per row n and
// one flag per timestep shared by all columns (rlcs_elig_trace_vec / _beta use the block kernel for
// few long rows): same kernel, the flag read per timestep instead of from a mask tile.
constexpr int kTmVec = 101;        // shared scalar decay
constexpr int kTmVecBeta = 102;    // decay per component and step in f1
constexpr int kTmVecBeta16 = 103;  // the same with 16 timesteps per warp and stage (see tm_rows)
__host__ __device__ constexpr bool tm_vec_beta(int a) { return a == kTmVecBeta || a == kTmVecBeta16; }
__host__ __device__ constexpr bool tm_row_mask(int a) { return a == kTmVec || tm_vec_beta(a); }
__host__ __device__ constexpr bool tm_forward(int a) { return a == kElig || a == kPrefix || tm_row_mask(a); }
// float tensors that are read at every step, and mask tensors
__host__ __device__ constexpr int tm_nf(int a) {
    return a == kRetrace ? 4 : a == kVtrace ? 3 : (a == kGae || a == kTdLambda || tm_vec_beta(a)) ? 2 : 1;
}
// timesteps per warp and stage in tm_block_kernel: fewer for Retrace, whose four float inputs make a
// row 576 bytes (measured: 0.84 -> 0.90 of the copy bandwidth with 4, while the lighter algorithms
// lose 5-12 % to the doubled per-stage overhead); more for the discounted return, whose rows are
// 160-192 bytes (0.52 -> 0.63 at 16384 environments with 16; the forward scans lose 1 % that way),
// and for the vector traces with the shared decay (128-byte rows; 0.63 -> 0.74 at 1024x1024x64 with
// 16, 0.61 with 32).  With a decay tensor 16 pay only while all blocks are resident at once (0.59 ->
// 0.76 at 512x2048x64, but 0.85 -> 0.77 at 1024x1024x64): two instances, chosen by the block count.
__host__ __device__ constexpr int tm_rows(int a) {
    return a == kRetrace ? 4 : (a == kDisc || a == kTmVec || a == kTmVecBeta16) ? 16 : 8;
}
__host__ __device__ constexpr int tm_row_bytes(int a, bool trunc) { return tm_nf(a) * 128 + (tm_row_mask(a) ? 0 : (trunc ? 2 : 1) * 32); }

// all ones where x != 0, else 0; written in PTX so that the flag reaches the arithmetic below as a
// plain word, not as a condition the compiler could branch on
__device__ __forceinline__ unsigned ones_if(unsigned x) {
    unsigned m;
    asm("{\n\t.reg .pred q;\n\tsetp.ne.u32 q, %1, 0;\n\tselp.u32 %0, 0xffffffff, 0, q;\n\t}" : "=r"(m) : "r"(x));
    return m;
}

// all ones where bit `pos` of x is set, else 0 (bfe.s32 sign-extends the one-bit field)
__device__ __forceinline__ unsigned bit_mask(unsigned x, int pos) {
    int m;
    asm("bfe.s32 %0, %1, %2, 1;" : "=r"(m) : "r"((int)x), "r"(pos));
    return (unsigned)m;
}

// predicated load: *ptr where m != 0 (the address is not touched otherwise), else 0
__device__ __forceinline__ float ldg_if_mask(const float* ptr, unsigned m) {
    float v = 0.f;
    asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.u32 q, %2, 0;\n\t@q ld.global.nc.f32 %0, [%1];\n\t}" : "+f"(v) : "l"(ptr), "r"(m));
    return v;
}

// m is all ones or all zero
__device__ __forceinline__ float keep(unsigned m, float x) { return __uint_as_float(__float_as_uint(x) & m); }
__device__ __forceinline__ float blend(unsigned m, float x1, float x0) {
    return __uint_as_float((__float_as_uint(x1) & m) | (__float_as_uint(x0) & ~m));
}

struct StepIn {
    float r, v1, v2, v3;   // the step's entries of f0..f3
    float bv;              // truncation continuation value; 0 unless the step is a live truncation
    unsigned dn, tr;       // mask bytes
};

struct BackState {
    float carry;      // recurrence value at t+1
    float prod;       // product of the betas walked so far (chunk aggregate)
    float v_next;     // V(s_{t+1}) | E_pi Q(s_{t+1},.) as stored in the buffer
    float lr_next;    // Retrace: log-ratio of step t+1
};

struct FwdState {
    float carry;      // recurrence value at t-1
    float prod;
    unsigned d_prev;  // dones flag of step t-1 (1 at t = 0: nothing to carry)
};

// Coefficients of one step, A_t = alpha + beta * A_{t+-1} (Table 1), plus V-trace's policy-gradient
// coefficient gamma * rho_t (0 where the step is cut).
struct Coef {
    float alpha, beta, pg;
};

// Backward algorithms, step t of one environment (Section 3.2 / 3.3).  Flags become all-ones /
// all-zero words and every choice is a bitwise blend: the flags differ from lane to lane, and a
// data-dependent branch would split the warp's 128-byte stores into partial ones.
template <int ALGO, bool TRUNC>
__device__ __forceinline__ Coef back_coef(const StepIn& in, const TmParams& p, unsigned last, float bootv, float v_next,
                                          float lr_next) {
    // last: all ones at the window's final step t = T-1, else 0
    // The step is cut (nothing is carried in) after a termination or a truncation: one test of both
    // flag bytes.  The successor value is then the truncation's continuation value -- in.bv, which
    // is 0 unless the step is a truncation that is not also a termination -- else the bootstrap at the
    // window edge, else the buffer's next entry.
    const unsigned cut = ones_if(TRUNC ? (in.dn | in.tr) : in.dn);
    const unsigned cont = ~(cut | last);
    const float succ = blend(cut, TRUNC ? in.bv : 0.f, blend(last, bootv, v_next));
    Coef c;
    c.pg = 0.f;
    if constexpr (ALGO == kGae) {
        c.alpha = fmaf(p.gamma, succ, in.r) - in.v1;
        c.beta = keep(cont, p.decay);
    } else if constexpr (ALGO == kTdLambda) {
        c.alpha = fmaf(blend(cont, p.aux, p.gamma), succ, in.r);
        c.beta = keep(cont, p.decay);
    } else if constexpr (ALGO == kDisc) {
        // a continued step has no successor term; succ is 0 there (no value tensor), so the blended
        // coefficient only matters where the step is cut
        c.alpha = fmaf(keep(~cont, p.gamma), succ, in.r);
        c.beta = keep(cont, p.decay);
    } else if constexpr (ALGO == kVtrace) {
        const float raw = expf(in.v3);
        const float rho = fminf(p.rho_bar, raw), cc = fminf(p.c_bar, raw);
        c.alpha = rho * (fmaf(p.gamma, succ, in.r) - in.v1);
        c.beta = keep(cont, p.gamma * cc);
        c.pg = keep(cont, p.gamma * rho);
    } else {   // kRetrace
        c.alpha = fmaf(p.gamma, succ, in.r) - in.v1;
        c.beta = keep(cont, p.aux * fminf(p.c_bar, expf(lr_next)));
    }
    return c;
}

// Forward algorithms (eligibility trace, episodic prefix sum): the carry into step t is severed by
// the flag of step t-1, or by the step's own flag where dones marks episode starts.
template <int ALGO>
__device__ __forceinline__ Coef fwd_coef(float x, unsigned d, unsigned d_prev, const TmParams& p, unsigned t) {
    const unsigned cutflag = (ALGO == kPrefix && p.starts_at) ? (t == 0 ? 1u : d) : d_prev;
    Coef c;
    c.alpha = x;
    c.beta = keep(~ones_if(cutflag), p.decay);
    c.pg = 0.f;
    return c;
}

// Outputs of one step from its recurrence value `val` and the scan-order predecessor's `prev`.
template <int ALGO>
__device__ __forceinline__ void emit(const TmParams& p, long long i, float val, float prev, float v1, const Coef& c) {
    if constexpr (ALGO == kGae) {
        __stcs(p.out0 + i, val);
        if (p.out1 != nullptr) __stcs(p.out1 + i, val + v1);
    } else if constexpr (ALGO == kVtrace) {
        __stcs(p.out0 + i, v1 + val);
        if (p.out1 != nullptr) __stcs(p.out1 + i, fmaf(c.pg, prev, c.alpha));
    } else if constexpr (ALGO == kRetrace) {
        __stcs(p.out0 + i, v1 + val);
    } else {
        __stcs(p.out0 + i, val);
    }
}

template <int ALGO, bool TRUNC, int MODE>
__device__ __forceinline__ void back_step(const StepIn& in, const TmParams& p, unsigned t, long long i, float bootv,
                                          bool write, BackState& st) {
    const Coef c = back_coef<ALGO, TRUNC>(in, p, (t == p.T - 1) ? ~0u : 0u, bootv, st.v_next, st.lr_next);
    const float val = fmaf(c.beta, st.carry, c.alpha);
    if (MODE != 1 && write) emit<ALGO>(p, i, val, st.carry, in.v1, c);
    st.carry = val;
    if (MODE == 1) st.prod *= c.beta;
    if constexpr (ALGO == kRetrace) {
        st.v_next = in.v2;
        st.lr_next = in.v3;
    } else if constexpr (tm_nf(ALGO) >= 2) {
        st.v_next = in.v1;
    }
}

template <int ALGO, int MODE>
__device__ __forceinline__ void fwd_step(float x, unsigned d, const TmParams& p, unsigned t, long long i, bool write,
                                         FwdState& st) {
    const Coef c = fwd_coef<ALGO>(x, d, st.d_prev, p, t);
    const float val = fmaf(c.beta, st.carry, c.alpha);
    if (MODE != 1 && write) emit<ALGO>(p, i, val, st.carry, 0.f, c);
    st.carry = val;
    if (MODE == 1) st.prod *= c.beta;
    st.d_prev = d;
}

// successor-side neighbours of a chunk's last step, when they lie inside the buffer
template <int ALGO>
__device__ __forceinline__ void init_back(BackState& st, const TmParams& p, long long n, unsigned t_hi, float carry) {
    st.carry = carry;
    st.prod = 1.f;
    st.v_next = 0.f;
    st.lr_next = 0.f;
    if (t_hi < p.T) {
        if constexpr (ALGO == kGae || ALGO == kTdLambda || ALGO == kVtrace) st.v_next = __ldg(p.f1 + (long long)t_hi * p.N + n);
        if constexpr (ALGO == kRetrace) {
            st.v_next = __ldg(p.f2 + (long long)t_hi * p.N + n);
            st.lr_next = __ldg(p.f3 + (long long)t_hi * p.N + n);
        }
    }
}

__device__ __forceinline__ void init_fwd(FwdState& st, const TmParams& p, long long n, unsigned t_lo, float carry) {
    st.carry = carry;
    st.prod = 1.f;
    st.d_prev = 1;
    if (t_lo > 0) st.d_prev = __ldg(p.dones + (long long)(t_lo - 1) * p.N + n);
}

// ---------------------------------------------------------------------------------------------
// Register path.  Steps of a chunk are numbered q = 0 .. len-1 in scan order.
// ---------------------------------------------------------------------------------------------

template <int ALGO, bool TRUNC>
struct Blk {
    StepIn s[kRows];
};

template <int ALGO>
__device__ __forceinline__ unsigned step_t(unsigned t_lo, unsigned t_hi, unsigned q) {
    return tm_forward(ALGO) ? t_lo + q : t_hi - 1 - q;
}

template <int ALGO, bool TRUNC>
__device__ __forceinline__ void load_blk(Blk<ALGO, TRUNC>& k, const TmParams& p, long long n, unsigned q0, unsigned len,
                                         unsigned t_lo, unsigned t_hi) {
#pragma unroll
    for (int u = 0; u < kRows; ++u) {
        if (q0 + u < len) {
            const long long i = (long long)step_t<ALGO>(t_lo, t_hi, q0 + u) * p.N + n;
            k.s[u].dn = __ldcs(p.dones + i);
            k.s[u].tr = TRUNC ? __ldcs(p.truncs + i) : 0u;
            k.s[u].r = __ldcs(p.f0 + i);
            if constexpr (tm_nf(ALGO) >= 2) k.s[u].v1 = __ldcs(p.f1 + i);
            if constexpr (ALGO == kRetrace) k.s[u].v2 = __ldcs(p.f2 + i);
            if constexpr (ALGO == kVtrace || ALGO == kRetrace) k.s[u].v3 = __ldcs(p.f3 + i);
        }
    }
}

// sparse truncation continuation values of a block whose masks have been loaded
template <int ALGO, bool TRUNC>
__device__ __forceinline__ void load_bv(Blk<ALGO, TRUNC>& k, const TmParams& p, long long n, unsigned q0, unsigned len,
                                        unsigned t_lo, unsigned t_hi) {
    if constexpr (TRUNC) {
#pragma unroll
        for (int u = 0; u < kRows; ++u) {
            k.s[u].bv = 0.f;
            if (q0 + u < len)
                k.s[u].bv = rlcs::ldg_if(p.trunc_boot + (long long)step_t<ALGO>(t_lo, t_hi, q0 + u) * p.N + n,
                                         k.s[u].tr != 0 && k.s[u].dn == 0);
        }
    }
}

template <int ALGO, bool TRUNC, int MODE>
__device__ __forceinline__ void walk_blk(const Blk<ALGO, TRUNC>& k, const TmParams& p, long long n, unsigned q0,
                                         unsigned len, unsigned t_lo, unsigned t_hi, float bootv, bool write,
                                         BackState& bs, FwdState& fs) {
#pragma unroll
    for (int u = 0; u < kRows; ++u) {
        if (q0 + u < len) {
            const unsigned t = step_t<ALGO>(t_lo, t_hi, q0 + u);
            const long long i = (long long)t * p.N + n;
            if constexpr (tm_forward(ALGO)) fwd_step<ALGO, MODE>(k.s[u].r, k.s[u].dn, p, t, i, write, fs);
            else back_step<ALGO, TRUNC, MODE>(k.s[u], p, t, i, bootv, write, bs);
        }
    }
}

// MODE 0: whole columns, write outputs.  MODE 1: chunk aggregates only.  MODE 2: walk from the
// chained carry and write outputs.
template <int ALGO, bool TRUNC, int MODE>
__global__ void __launch_bounds__(kThreads) tm_kernel(const TmParams p) {
    constexpr bool FWD = tm_forward(ALGO);
    const long long n_raw = (long long)blockIdx.x * kThreads + threadIdx.x;
    const bool write = n_raw < p.N;                          // lanes past N shadow the last column
    const long long n = write ? n_raw : p.N - 1;
    const unsigned k = blockIdx.y;
    const unsigned t_lo = k * p.chunk;
    const unsigned t_hi = min(p.T, t_lo + p.chunk);          // chunk = [t_lo, t_hi)
    const unsigned len = t_hi - t_lo;
    const float bootv = (!FWD && p.boot != nullptr) ? __ldg(p.boot + n) : 0.f;
    const float carry0 = MODE == 2 ? p.agg_a[(long long)k * p.N + n] : 0.f;

    BackState bs = {};
    FwdState fs = {};
    if constexpr (FWD) init_fwd(fs, p, n, t_lo, carry0);
    else init_back<ALGO>(bs, p, n, t_hi, carry0);

    // Two register sets alternate: while one block of kRows steps is walked, the loads of the next one
    // are in flight, and its truncation values are requested as soon as its masks have arrived.  The
    // __syncwarp() calls are there for speed, not for correctness: lanes that drift apart (the sparse
    // predicated loads finish at different times) are not brought back together by the hardware, and
    // a split warp turns every 128-byte row into several partial accesses.
    Blk<ALGO, TRUNC> a, b;
    unsigned q = 0;
    load_blk<ALGO, TRUNC>(a, p, n, q, len, t_lo, t_hi);
    load_bv<ALGO, TRUNC>(a, p, n, q, len, t_lo, t_hi);
    for (;;) {
        __syncwarp();
        if (q + kRows < len) load_blk<ALGO, TRUNC>(b, p, n, q + kRows, len, t_lo, t_hi);
        walk_blk<ALGO, TRUNC, MODE>(a, p, n, q, len, t_lo, t_hi, bootv, write, bs, fs);
        q += kRows;
        if (q >= len) break;
        load_bv<ALGO, TRUNC>(b, p, n, q, len, t_lo, t_hi);
        __syncwarp();
        if (q + kRows < len) load_blk<ALGO, TRUNC>(a, p, n, q + kRows, len, t_lo, t_hi);
        walk_blk<ALGO, TRUNC, MODE>(b, p, n, q, len, t_lo, t_hi, bootv, write, bs, fs);
        q += kRows;
        if (q >= len) break;
        load_bv<ALGO, TRUNC>(a, p, n, q, len, t_lo, t_hi);
    }
    if (MODE == 1 && write) {
        p.agg_a[(long long)k * p.N + n] = FWD ? fs.carry : bs.carry;
        p.agg_b[(long long)k * p.N + n] = FWD ? fs.prod : bs.prod;
    }
}

// ---------------------------------------------------------------------------------------------
// Staged path: per-warp shared-memory ring filled by cp.async.
// ---------------------------------------------------------------------------------------------

// 16-byte asynchronous copy global -> shared through L2 only; bytes = 0 fills the 16 bytes with zeros
__device__ __forceinline__ void cp_async16(void* dst_smem, const void* src, unsigned bytes) {
    const unsigned d = (unsigned)__cvta_generic_to_shared(dst_smem);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(d), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
// wait until at most `pending` of this thread's committed groups are still in flight
__device__ __forceinline__ void cp_async_wait(int pending) {
    switch (pending) {
        case 0: asm volatile("cp.async.wait_group 0;" ::: "memory"); break;
        case 1: asm volatile("cp.async.wait_group 1;" ::: "memory"); break;
        case 2: asm volatile("cp.async.wait_group 2;" ::: "memory"); break;
        case 3: asm volatile("cp.async.wait_group 3;" ::: "memory"); break;
        case 4: asm volatile("cp.async.wait_group 4;" ::: "memory"); break;
        case 5: asm volatile("cp.async.wait_group 5;" ::: "memory"); break;
        case 6: asm volatile("cp.async.wait_group 6;" ::: "memory"); break;
        case 7: asm volatile("cp.async.wait_group 7;" ::: "memory"); break;
        case 8: asm volatile("cp.async.wait_group 8;" ::: "memory"); break;
        case 9: asm volatile("cp.async.wait_group 9;" ::: "memory"); break;
        case 10: asm volatile("cp.async.wait_group 10;" ::: "memory"); break;
        case 11: asm volatile("cp.async.wait_group 11;" ::: "memory"); break;
        case 12: asm volatile("cp.async.wait_group 12;" ::: "memory"); break;
        case 13: asm volatile("cp.async.wait_group 13;" ::: "memory"); break;
        case 14: asm volatile("cp.async.wait_group 14;" ::: "memory"); break;
        case 15: asm volatile("cp.async.wait_group 15;" ::: "memory"); break;
        default: asm volatile("cp.async.wait_group 0;" ::: "memory"); break;   // waits for more than asked: still correct
    }
}

constexpr int kMaxStages = 16;

// One stage of a thread block: R = KR * warps rows (KR = tm_rows(ALGO) timesteps per warp) of its 32 C columns (C columns per lane), row
// index = scan-order step within the stage.  Floats and masks live in separate rings (the mask ring
// runs two stages ahead): float tensor a at fbase[a][row][32 C floats], mask tensor m at
// mbase[m][row][32 C bytes].
template <int ALGO, bool TRUNC, int W, int C>
struct StageView {
    static constexpr int NF = tm_nf(ALGO);
    static constexpr int NM = tm_row_mask(ALGO) ? 0 : (TRUNC ? 2 : 1);
    static constexpr int KR = tm_rows(ALGO);
    static constexpr int R = KR * W;
    unsigned char* fbase;
    unsigned char* mbase;
    __device__ __forceinline__ float* f(int a, int row) const { return reinterpret_cast<float*>(fbase + (a * R + row) * (128 * C)); }
    __device__ __forceinline__ uint8_t* m(int a, int row) const { return mbase + (a * R + row) * (32 * C); }
};

// A lane's C adjacent values of one row
template <int C>
__device__ __forceinline__ void lds_f(const float* row, int lane, float (&x)[C]) {
    if constexpr (C == 2) { const float2 v = *reinterpret_cast<const float2*>(row + 2 * lane); x[0] = v.x; x[1] = v.y; }
    else x[0] = row[lane];
}
template <int C>
__device__ __forceinline__ void lds_m(const uint8_t* row, int lane, unsigned (&x)[C]) {
    if constexpr (C == 2) { const unsigned v = *reinterpret_cast<const unsigned short*>(row + 2 * lane); x[0] = v & 0xffu; x[1] = v >> 8; }
    else x[0] = row[lane];
}
template <int C>
__device__ __forceinline__ void sts_f(float* row, int lane, const float (&x)[C]) {
    if constexpr (C == 2) *reinterpret_cast<float2*>(row + 2 * lane) = make_float2(x[0], x[1]);
    else row[lane] = x[0];
}
template <int C>
__device__ __forceinline__ void stg_f(float* p, const float (&x)[C]) {
    if constexpr (C == 2) __stcs(reinterpret_cast<float2*>(p), make_float2(x[0], x[1]));
    else __stcs(p, x[0]);
}

// Per-thread bookkeeping for the copies of a stage.  A row of a float tensor is 8 C 16-byte pieces,
// a row of a mask tensor 2 C; a thread moves the same piece of 2 C float rows and of one mask row
// per stage.  Rows past the chunk and pieces past column N are zero-filled (N is a multiple of 16
// here, so a piece is never split by the edge).
struct CopyPlan {
    long long i_first;     // flat index of the chunk's scan-order step 0, first column of the block
    long long rowstep;     // flat-index step between scan-order neighbours: +N forward, -N backward
    unsigned len;          // steps in the chunk
    int frow, fcol;        // first float row of this thread, column offset of its piece
    bool fcol_ok;
    int mrow, mcol;
    bool m_on;
};

template <int ALGO, bool TRUNC, int W, int C>
__device__ __forceinline__ void issue_floats(const StageView<ALGO, TRUNC, W, C>& sv, const TmParams& p, const CopyPlan& cp, unsigned s) {
    constexpr int KR = tm_rows(ALGO);
    constexpr int R = KR * W;
    const float* const fsrc[4] = {p.f0, p.f1, p.f2, p.f3};
    constexpr int fidx[4] = {0, 1, (ALGO == kVtrace) ? 3 : 2, 3};   // V-trace stages f0, f1, f3
#pragma unroll
    for (int h = 0; h < KR * C / 4; ++h) {
        const int row = cp.frow + h * (4 * W / C);
        const unsigned q = s * R + row;
        const bool ok = cp.fcol_ok && q < cp.len;
        const long long off = ok ? cp.i_first + cp.rowstep * q + cp.fcol : 0;
#pragma unroll
        for (int a = 0; a < tm_nf(ALGO); ++a)
            cp_async16(sv.f(a, row) + cp.fcol, fsrc[fidx[a]] + off, ok ? 16u : 0u);
    }
}

template <int ALGO, bool TRUNC, int W, int C>
__device__ __forceinline__ void issue_masks(const StageView<ALGO, TRUNC, W, C>& sv, const TmParams& p, const CopyPlan& cp, unsigned s) {
    if constexpr (tm_row_mask(ALGO)) return;
    if (cp.m_on) {
        const unsigned q = s * (tm_rows(ALGO) * W) + cp.mrow;
        const bool ok = q < cp.len;
        const long long off = ok ? cp.i_first + cp.rowstep * q + cp.mcol : 0;
        cp_async16(sv.m(0, cp.mrow) + cp.mcol, p.dones + off, ok ? 16u : 0u);
        if constexpr (TRUNC) cp_async16(sv.m(1, cp.mrow) + cp.mcol, p.truncs + off, ok ? 16u : 0u);
    }
}

// Which of a warp's KR rows of a stage hold a set flag: the rows are KR * 32 C adjacent bytes of the
// mask ring, every lane takes KR C of them (32 / KR lanes per row) and one ballot shares the answer.
// Bit 32 / KR * u + x: lane x's share of row u has a nonzero byte.  All 32 lanes must call.
template <int KR, int C>
__device__ __forceinline__ unsigned row_flag_bits(const uint8_t* rows, int lane) {
    constexpr int B = KR * C;
    static_assert(B == 4 || B == 8 || B == 16 || B == 32, "a lane's share is one or two vector loads");
    unsigned any;
    if constexpr (B == 4) {
        any = *reinterpret_cast<const unsigned*>(rows + 4 * lane);
    } else if constexpr (B == 8) {
        const uint2 v = *reinterpret_cast<const uint2*>(rows + 8 * lane);
        any = v.x | v.y;
    } else {
        any = 0;
#pragma unroll
        for (int h = 0; h < B / 16; ++h) {
            const uint4 v = *reinterpret_cast<const uint4*>(rows + B * lane + 16 * h);
            any |= v.x | v.y | v.z | v.w;
        }
    }
    return __ballot_sync(0xffffffffu, any != 0);
}
template <int KR>
__device__ __forceinline__ bool row_flagged(unsigned bits, int u) {
    constexpr int L = 32 / KR;
    return ((bits >> (L * u)) & ((1u << L) - 1u)) != 0;
}

// truncation continuation values of `nvalid` rows from row0 of a stage whose masks have landed;
// i = flat index of the first of them for this lane's first column.  With flags as rare as they are
// most rows of 32 C columns hold no truncation at all: those are skipped on a warp-uniform test
// (no divergence), and only the others read their flags lane by lane.
template <int ALGO, bool TRUNC, int W, int C>
__device__ __forceinline__ void stage_bv(float (&bv)[tm_rows(ALGO)][C], const StageView<ALGO, TRUNC, W, C>& sv, const TmParams& p,
                                         long long i, int rowbytes, int row0, int nvalid, int lane, unsigned write_mask) {
    constexpr int KR = tm_rows(ALGO);
    if (nvalid <= 0) return;                                 // past the chunk: the values are never used
    const unsigned trbits = row_flag_bits<KR, C>(sv.m(1, row0), lane);
#pragma unroll
    for (int u = 0; u < KR; ++u)
#pragma unroll
        for (int c = 0; c < C; ++c) bv[u][c] = 0.f;
    if (trbits == 0) return;
#pragma unroll
    for (int u = 0; u < KR; ++u) {
        if (row_flagged<KR>(trbits, u)) {
            unsigned tr[C], dn[C];
            lds_m<C>(sv.m(1, row0 + u), lane, tr);
            lds_m<C>(sv.m(0, row0 + u), lane, dn);
            const unsigned rowmask = write_mask & (u < nvalid ? ~0u : 0u);
            // rowbytes * u is one multiply-add onto the 64-bit address (u is a constant here)
            const float* const src = reinterpret_cast<const float*>(reinterpret_cast<const char*>(p.trunc_boot + i) + (long long)rowbytes * u);
#pragma unroll
            for (int c = 0; c < C; ++c) bv[u][c] = ldg_if_mask(src + c, ones_if(tr[c]) & ~ones_if(dn[c]) & rowmask);
        }
    }
}

__device__ __forceinline__ int wrap_next(int x, int n) { return x + 1 == n ? 0 : x + 1; }
__device__ __forceinline__ int wrap_prev(int x, int n) { return x == 0 ? n - 1 : x - 1; }

// A thread block owns 32 C adjacent environments (a lane C of them: with C = 2 every shared-memory
// read, store and address computation serves two steps); its W warps split every stage of
// R = KR * W timesteps in time (KR = tm_rows).  Per stage: each warp walks its KR steps from carry 0, keeping
// per step the value so far and the running product of betas (the step's affine map of the incoming
// carry, Eq. 2); the W per-warp aggregates go through shared memory; every warp folds them in scan
// order onto the block's carry (a few FMAs, redundantly in each warp) to get its own incoming
// carry, and finishes its steps with one FMA each.  The inputs cross HBM once however the time
// axis is split.
//
// Copies are committed in groups {floats of stage s, masks of stage s+2}: when a stage's floats
// have landed so have the masks two stages on, and the sparse truncation values they point at are
// requested two stages before their use (registers bv1, bv2).  One stage is not enough: with the
// ring's 16 MB in flight a load takes 2.5 us or more to come back, a stage lasts under 2 (measured:
// GAE 0.80 -> 0.65 of the copy bandwidth at 16384 x 2048 with a distance of one stage).
// MODE as in tm_kernel, plus MODE 3 for the chained kernel of the vector traces (one flag per
// timestep, so a cut holds for all columns at once): the walk starts from carry 0; the steps from the
// first cut on do not depend on the chunk's incoming carry and are written as in MODE 0; the
// `qdefer` steps before it are not written -- their value from carry 0 replaces the step's f0 entry in
// the ring (which only its own thread reads) and, with a decay tensor, the product of the betas from
// the chunk's first step up to and including it replaces the f1 entry -- so that the caller can finish
// them once the carry is known, without walking the chunk again.  The ring must then hold the whole
// chunk (stages >= the chunk's stage count, no slot refilled).
// block_walk: chunk k of the block's 32 C columns from n0.  A: in, the carry into the chunk (MODE 0: 0;
// MODE 1: 0); out, the recurrence value after the chunk's last step.  P: out, the product of the
// chunk's betas.  Every thread returns the values of its own columns.
template <int ALGO, bool TRUNC, int MODE, int W, int C>
__device__ __forceinline__ void block_walk(const TmParams& p, const long long n0, const unsigned k, float (&A)[C], float (&P)[C],
                                           const unsigned qdefer = 0) {
    constexpr bool FWD = tm_forward(ALGO);
    constexpr bool ROWMASK = tm_row_mask(ALGO);
    using SV = StageView<ALGO, TRUNC, W, C>;
    extern __shared__ __align__(16) unsigned char tm_smem[];
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    constexpr int KR = tm_rows(ALGO);
    constexpr int R = KR * W;
    const int S = p.stages, SM = S + 2;
    constexpr int fstage = R * SV::NF * 128 * C, mstage = R * SV::NM * 32 * C;
    unsigned char* const mring = tm_smem + (size_t)S * fstage;
    float2* const agg = reinterpret_cast<float2*>(mring + (size_t)SM * mstage);         // [2][W][32 C]
    float* const edge_v = reinterpret_cast<float*>(agg + 2 * W * 32 * C);               // [2][32 C]
    float* const edge_x = edge_v + 64 * C;                                              // [2][32 C] log-ratio | dones flag

    const bool write = n0 + C * lane < p.N;                  // lanes past N read zero-filled columns (N is even)
    const unsigned write_mask = write ? ~0u : 0u;
    const unsigned t_lo = k * p.chunk;
    const unsigned t_hi = min(p.T, t_lo + p.chunk);
    const unsigned len = t_hi - t_lo;
    const unsigned nst = (len + R - 1) / R;
    const unsigned edge_last = (!FWD && t_hi == p.T) ? ~0u : 0u;   // the chunk's first step in scan order is t = T-1

    CopyPlan cp;
    cp.rowstep = FWD ? p.N : -p.N;
    cp.i_first = (long long)(FWD ? t_lo : t_hi - 1) * p.N + n0;
    cp.len = len;
    cp.frow = tid / (8 * C); cp.fcol = 4 * (tid % (8 * C)); cp.fcol_ok = n0 + cp.fcol < p.N;
    cp.mrow = tid / (2 * C); cp.mcol = 16 * (tid % (2 * C)); cp.m_on = n0 + cp.mcol < p.N;

    // block state per column: the affine map of everything walked so far applied to the chunk's incoming carry;
    // neighbours across the chunk's scan-order start
    float bootv[C], v0[C], lr0[C];
    unsigned d0[C];
#pragma unroll
    for (int c = 0; c < C; ++c) {
        const long long n = write ? n0 + C * lane + c : p.N - 1;
        P[c] = 1.f;
        bootv[c] = (!FWD && p.boot != nullptr) ? __ldg(p.boot + n) : 0.f;
        BackState b0 = {};
        FwdState f0 = {};
        if constexpr (ROWMASK) f0.d_prev = 0;
        else if constexpr (FWD) init_fwd(f0, p, n, t_lo, 0.f);
        else init_back<ALGO>(b0, p, n, t_hi, 0.f);
        v0[c] = b0.v_next; lr0[c] = b0.lr_next; d0[c] = f0.d_prev;
    }

    // A group is committed for every stage index, empty past the end, so that "all but the newest P
    // groups" always names the same stages.  Floats of stage s sit in slot s mod S, masks in slot
    // s mod (S + 2).  With C = 1 only the first half of the threads has a mask piece.
    const bool mask_thread = tid < 2 * C * R;
    cp.m_on = cp.m_on && mask_thread;
    for (int s = 0; s + 1 < S; ++s) {
        if (s == 0) {
            if (0 < nst) issue_masks<ALGO, TRUNC>(SV{nullptr, mring}, p, cp, 0);
            if (1 < nst) issue_masks<ALGO, TRUNC>(SV{nullptr, mring + mstage}, p, cp, 1);
        }
        if ((unsigned)s < nst) issue_floats<ALGO, TRUNC>(SV{tm_smem + s * fstage, nullptr}, p, cp, s);
        if ((unsigned)s + 2 < nst) issue_masks<ALGO, TRUNC>(SV{nullptr, mring + (s + 2) * mstage}, p, cp, s + 2);
        cp_async_commit();
    }
    float bvc[KR][C], bv1[KR][C], bv2[KR][C];
#pragma unroll
    for (int u = 0; u < KR; ++u)
#pragma unroll
        for (int c = 0; c < C; ++c) bvc[u][c] = bv1[u][c] = bv2[u][c] = 0.f;
    const int row0 = KR * w;
    // this lane's flat index (first column) at its first row of the current stage, and rows it has there
    long long iw = cp.i_first + cp.rowstep * row0 + C * lane;
    int left = (int)len - row0;                              // steps from this warp's first row to the chunk's end
    const long long stagestep = cp.rowstep * R;
    const int rowbytes = (int)(cp.rowstep * 4);              // |N| * 4 fits: the host routes larger N to tm_kernel
    const bool all_write = __all_sync(0xffffffffu, write);
    if constexpr (TRUNC) {
        cp_async_wait(S - 2);                                // stage 0 and the masks of stages 0..2 have landed
        __syncthreads();
        stage_bv<ALGO, TRUNC>(bvc, SV{nullptr, mring}, p, iw, rowbytes, row0, left, lane, write_mask);
        stage_bv<ALGO, TRUNC>(bv1, SV{nullptr, mring + mstage}, p, iw + stagestep, rowbytes, row0, left - R, lane, write_mask);
    }
    int fs = 0, ms = 0;                                      // ring slots of stage j
    for (unsigned j = 0; j < nst; ++j) {
        const int par = j & 1;
        cp_async_wait(S - 2);                                // this thread's pieces of stage j (masks: j+2)
        __syncthreads();                                     // ... and everyone else's
        const SV cur{tm_smem + fs * fstage, mring + ms * mstage};
        const int nvalid = left < KR ? (left < 0 ? 0 : left) : KR;
        if constexpr (TRUNC) {
            const int ms2 = ms + 2 >= SM ? ms + 2 - SM : ms + 2;
            stage_bv<ALGO, TRUNC>(bv2, SV{nullptr, mring + ms2 * mstage}, p, iw + 2 * stagestep, rowbytes, row0, left - 2 * R,
                                  lane, write_mask);
        }
        // neighbour of this warp's first step: the row before it in the stage, the last row of the
        // previous stage, or the chunk's outside neighbour
        float v_next[C], lr_next[C];
        unsigned d_prev[C];
#pragma unroll
        for (int c = 0; c < C; ++c) { v_next[c] = 0.f; lr_next[c] = 0.f; d_prev[c] = 0; }
        if constexpr (ROWMASK) {
            // the flag of step t-1 is read per step below
        } else if (w > 0) {
            if constexpr (FWD) lds_m<C>(cur.m(0, row0 - 1), lane, d_prev);
            else if constexpr (ALGO == kRetrace) { lds_f<C>(cur.f(2, row0 - 1), lane, v_next); lds_f<C>(cur.f(3, row0 - 1), lane, lr_next); }
            else if constexpr (SV::NF >= 2) lds_f<C>(cur.f(1, row0 - 1), lane, v_next);
        } else if (j > 0) {
            float t[C];
            if constexpr (FWD) {
                lds_f<C>(edge_x + (par ^ 1) * 32 * C, lane, t);
#pragma unroll
                for (int c = 0; c < C; ++c) d_prev[c] = __float_as_uint(t[c]);
            } else {
                lds_f<C>(edge_v + (par ^ 1) * 32 * C, lane, v_next);
                lds_f<C>(edge_x + (par ^ 1) * 32 * C, lane, lr_next);
            }
        } else {
#pragma unroll
            for (int c = 0; c < C; ++c) { v_next[c] = v0[c]; lr_next[c] = lr0[c]; d_prev[c] = d0[c]; }
        }
        // pass 1: from carry 0
        float val0[KR][C], pb[KR][C], v1[KR][C], pgc[KR][C], alp[KR][C];
        float carry[C], prod[C];
#pragma unroll
        for (int c = 0; c < C; ++c) { carry[c] = 0.f; prod[c] = 1.f; }
        // the per-row guards exist only in the instance that the chunk's ragged last stage takes
        // one flag per timestep: the flags of the steps before this warp's rows (cut into step t <=> t == 0 or dones[t-1])
        // bit u: the carry into this warp's row u is cut.  Lane u reads the flag; one ballot shares them.
        unsigned cutbits = 0;
        if constexpr (ROWMASK) {
            static_assert(KR <= 32, "one lane per row of the warp");
            const unsigned t = t_lo + j * R + row0 + lane;
            unsigned f = 1u;
            if (lane < KR && t != 0 && t <= p.T) f = __ldg(p.dones + t - 1);
            cutbits = __ballot_sync(0xffffffffu, f != 0);
        }
        auto pass1 = [&](auto full) {
            constexpr bool FULL = decltype(full)::value;
#pragma unroll
            for (int u = 0; u < KR; ++u) {
#pragma unroll
                for (int c = 0; c < C; ++c) { v1[u][c] = 0.f; pgc[u][c] = 0.f; alp[u][c] = 0.f; }
                if (FULL || u < nvalid) {
                    float r[C], x1[C], x2[C], x3[C];
                    unsigned dn[C], tr[C];
                    lds_f<C>(cur.f(0, row0 + u), lane, r);
                    if constexpr (ROWMASK) {
                        if constexpr (tm_vec_beta(ALGO)) lds_f<C>(cur.f(1, row0 + u), lane, x1);
#pragma unroll
                        for (int c = 0; c < C; ++c) dn[c] = 0;
                    } else {
                        lds_m<C>(cur.m(0, row0 + u), lane, dn);
                    }
                    if constexpr (!FWD) {
                        if constexpr (SV::NF >= 2) lds_f<C>(cur.f(1, row0 + u), lane, x1);
                        if constexpr (ALGO == kRetrace) { lds_f<C>(cur.f(2, row0 + u), lane, x2); lds_f<C>(cur.f(3, row0 + u), lane, x3); }
                        if constexpr (ALGO == kVtrace) lds_f<C>(cur.f(2, row0 + u), lane, x3);
                        if constexpr (TRUNC) lds_m<C>(cur.m(1, row0 + u), lane, tr);
                    }
#pragma unroll
                    for (int c = 0; c < C; ++c) {
                        Coef co;
                        if constexpr (ROWMASK) {
                            co.alpha = r[c];
                            co.beta = keep(~bit_mask(cutbits, u), tm_vec_beta(ALGO) ? x1[c] : p.decay);
                            co.pg = 0.f;
                        } else if constexpr (FWD) {
                            co = fwd_coef<ALGO>(r[c], dn[c], d_prev[c], p, (u == 0 && w == 0 && j == 0) ? t_lo : 1u);
                            d_prev[c] = dn[c];
                        } else {
                            StepIn in;
                            in.r = r[c];
                            in.v1 = SV::NF >= 2 ? x1[c] : 0.f;
                            in.v2 = ALGO == kRetrace ? x2[c] : 0.f;
                            in.v3 = (ALGO == kRetrace || ALGO == kVtrace) ? x3[c] : 0.f;
                            in.dn = dn[c];
                            in.tr = TRUNC ? tr[c] : 0u;
                            in.bv = bvc[u][c];
                            // only the block's very first row can be the window's final step
                            const unsigned last = (u == 0 && w == 0 && j == 0) ? edge_last : 0u;
                            co = back_coef<ALGO, TRUNC>(in, p, last, bootv[c], v_next[c], lr_next[c]);
                            v_next[c] = ALGO == kRetrace ? in.v2 : in.v1;
                            lr_next[c] = in.v3;
                            v1[u][c] = in.v1;
                        }
                        carry[c] = fmaf(co.beta, carry[c], co.alpha);
                        prod[c] *= co.beta;
                        pgc[u][c] = co.pg;
                        alp[u][c] = co.alpha;
                    }
                }
#pragma unroll
                for (int c = 0; c < C; ++c) { val0[u][c] = carry[c]; pb[u][c] = prod[c]; }
            }
        };
        if (nvalid == KR) pass1(std::true_type{});
        else pass1(std::false_type{});
#pragma unroll
        for (int c = 0; c < C; ++c) agg[((par * W + w) * 32 + lane) * C + c] = make_float2(carry[c], prod[c]);
        if (!ROWMASK && w == W - 1) {                        // neighbours for the next stage's first warp
#pragma unroll
            for (int c = 0; c < C; ++c) {
                if constexpr (FWD) edge_x[par * 32 * C + C * lane + c] = __uint_as_float(d_prev[c]);
                else { edge_v[par * 32 * C + C * lane + c] = v_next[c]; edge_x[par * 32 * C + C * lane + c] = lr_next[c]; }
            }
        }
        __syncthreads();
        // fold the warps' aggregates in scan order onto the block state
        float cin[C], pin[C];                                // value and beta product at the entry of this warp's rows
#pragma unroll
        for (int c = 0; c < C; ++c) { cin[c] = A[c]; pin[c] = P[c]; }
#pragma unroll
        for (int x = 0; x < W; ++x) {
#pragma unroll
            for (int c = 0; c < C; ++c) {
                const float2 ab = agg[((par * W + x) * 32 + lane) * C + c];
                if (x == w) { cin[c] = A[c]; if (MODE == 3 && tm_vec_beta(ALGO)) pin[c] = P[c]; }
                A[c] = fmaf(ab.y, A[c], ab.x);
                P[c] *= ab.y;
            }
        }
        // pass 2: one FMA per step, then the outputs.  The common case -- every row of the warp inside the
        // chunk, every lane inside N -- has no guard at all; whether there is a second output tensor is
        // decided once per stage, not per store.
        if (MODE != 1) {
            auto pass2 = [&](auto full, auto both) {
                constexpr bool FULL = decltype(full)::value;
                constexpr bool BOTH = decltype(both)::value;
                float prev[C];
#pragma unroll
                for (int c = 0; c < C; ++c) prev[c] = cin[c];
                char* const dst0 = reinterpret_cast<char*>(p.out0 + iw);
                char* const dst1 = BOTH ? reinterpret_cast<char*>(p.out1 + iw) : nullptr;
#pragma unroll
                for (int u = 0; u < KR; ++u) {
                    if (FULL || (u < nvalid && write)) {
                        float o0[C], o1[C];
#pragma unroll
                        for (int c = 0; c < C; ++c) {
                            const float val = fmaf(pb[u][c], cin[c], val0[u][c]);
                            if constexpr (ALGO == kGae) { o0[c] = val; o1[c] = val + v1[u][c]; }
                            else if constexpr (ALGO == kVtrace) { o0[c] = v1[u][c] + val; o1[c] = fmaf(pgc[u][c], prev[c], alp[u][c]); }
                            else if constexpr (ALGO == kRetrace) { o0[c] = v1[u][c] + val; o1[c] = 0.f; }
                            else { o0[c] = val; o1[c] = 0.f; }
                            prev[c] = val;
                        }
                        if (MODE == 3 && j * R + row0 + u < qdefer) {      // (uniform over the warp)
                            sts_f<C>(cur.f(0, row0 + u), lane, o0);
                            if constexpr (tm_vec_beta(ALGO)) {
                                float sens[C];
#pragma unroll
                                for (int c = 0; c < C; ++c) sens[c] = pb[u][c] * pin[c];
                                sts_f<C>(cur.f(1, row0 + u), lane, sens);
                            }
                        } else {
                            stg_f<C>(reinterpret_cast<float*>(dst0 + (long long)rowbytes * u), o0);
                            if constexpr (BOTH) stg_f<C>(reinterpret_cast<float*>(dst1 + (long long)rowbytes * u), o1);
                        }
                    }
                }
            };
            const bool fast = nvalid == KR && all_write;
            if constexpr (ALGO == kGae || ALGO == kVtrace) {
                if (p.out1 != nullptr) {
                    if (fast) pass2(std::true_type{}, std::true_type{});
                    else pass2(std::false_type{}, std::true_type{});
                } else {
                    if (fast) pass2(std::true_type{}, std::false_type{});
                    else pass2(std::false_type{}, std::false_type{});
                }
            } else {
                if (fast) pass2(std::true_type{}, std::false_type{});
                else pass2(std::false_type{}, std::false_type{});
            }
        }
        // everyone is past the barrier, hence done with stage j-1: refill its slots
        {
            const unsigned s = j + S - 1;
            if (s < nst) issue_floats<ALGO, TRUNC>(SV{tm_smem + wrap_prev(fs, S) * fstage, nullptr}, p, cp, s);
            if (s + 2 < nst) issue_masks<ALGO, TRUNC>(SV{nullptr, mring + wrap_prev(ms, SM) * mstage}, p, cp, s + 2);
            cp_async_commit();
        }
#pragma unroll
        for (int u = 0; u < KR; ++u)
#pragma unroll
            for (int c = 0; c < C; ++c) { bvc[u][c] = bv1[u][c]; bv1[u][c] = bv2[u][c]; }
        fs = wrap_next(fs, S);
        ms = wrap_next(ms, SM);
        iw += stagestep;
        left -= R;
    }
    cp_async_wait(0);
}

// this block's problem of a batch (vector traces: row z)
template <int ALGO>
__device__ __forceinline__ TmParams batch_slice(const TmParams& p_in, unsigned z) {
    TmParams p = p_in;
    if constexpr (tm_row_mask(ALGO)) {
        const long long off = (long long)z * p_in.batch_stride;
        p.f0 += off;
        if constexpr (tm_vec_beta(ALGO)) p.f1 += off;
        p.out0 += off;
        p.dones += (long long)z * p_in.T;
    }
    return p;
}

// (No register cap: holding these kernels to the 80 registers that six 128-thread blocks per SM would
// need was measured and loses -- the discounted return spills and halves, V-trace and Retrace lose
// 0.03-0.10 of the copy bandwidth -- although the ring is planned for up to six blocks.)
template <int ALGO, bool TRUNC, int MODE, int W, int C>
__global__ void __launch_bounds__(32 * W) tm_block_kernel(const TmParams p_in) {
    // (no-ops unless launched with programmatic stream serialisation: then the blocks may be placed
    // while the kernel before this one drains, and nothing in global memory is touched before it is done)
    rlcs::grid_dependency_launch();
    rlcs::grid_dependency_wait();
    const TmParams p = batch_slice<ALGO>(p_in, blockIdx.z);
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const long long n0 = (long long)blockIdx.x * (32 * C);
    const unsigned k = blockIdx.y;
    const bool write = n0 + C * lane < p.N;
    float A[C], P[C];
#pragma unroll
    for (int c = 0; c < C; ++c) A[c] = (MODE == 2 && write) ? p.agg_a[(long long)k * p.N + n0 + C * lane + c] : 0.f;
    block_walk<ALGO, TRUNC, MODE, W, C>(p, n0, k, A, P);
    if (MODE == 1 && write && w == 0) {
#pragma unroll
        for (int c = 0; c < C; ++c) {
            p.agg_a[(long long)k * p.N + n0 + C * lane + c] = A[c];
            p.agg_b[(long long)k * p.N + n0 + C * lane + c] = P[c];
        }
    }
}

// The time axis cut without a second read from HBM and without a second walk: one launch, every block
// takes a (column block, chunk) pair from a ticket counter -- chunk index slowest, so that the
// scan-order predecessors of a chunk hold lower tickets and are running or done when it starts --
// walks its chunk once from carry 0, writing the outputs that result and leaving every step's
// sensitivity to the incoming carry in the ring (block_walk, MODE 3), publishes the aggregate
// (A, P) = (value after the last step from carry 0, product of betas), looks back for the carry c
// into its chunk, publishes the value it carries out, and adds sensitivity * c to the outputs of the
// steps that c reaches: those before the chunk's first cut, a fifth of the chunk at the recipe's
// flag rate, read back from L2 where the block wrote them moments before.
//
// Records are 16 bytes {value, kind, beta product, kind}, kind 0 = not yet (the call zeroes them),
// 1 = aggregate, 2 = carried-out value; each 8-byte half carries the kind, so a record read while it
// changes shows two different kinds and is read again.  The carry into chunk s is by definition the
// left fold v_j = fma(P_j, v_{j-1}, A_j) over its predecessors; the look-back walks back to the
// nearest record that fixes a value without its own predecessor (kind 2, P = 0, or chunk 0) and
// re-applies the aggregates after it in that same order, so the result does not depend on timing.
// Waits are bounded: after spin_cap polls of one record the status word is set and the carry taken as 0.
constexpr int kLookbackDepth = 16;     // aggregates remembered before waiting for a carried-out value

__device__ __forceinline__ float chained_carry(const TmParams& p, long long rec0, unsigned ks) {
    // rec0: record of scan-order chunk 0 for this column; records of later chunks follow every npad
    float sa[kLookbackDepth], sb[kLookbackDepth];
    int n = 0;
    long long j = (long long)ks - 1;
    unsigned polls = 0;
    float start = 0.f;
    for (;;) {
        const uint4 v = rlcs::ld_volatile_u4(p.records + rec0 + j * p.npad);
        const float a = __uint_as_float(v.x), b = __uint_as_float(v.z);
        const bool ready = v.y == v.w && v.y != 0;
        if (ready && (v.y == 2 || b == 0.f || j == 0)) { start = a; break; }
        if (ready && n < kLookbackDepth) { sa[n] = a; sb[n] = b; ++n; --j; polls = 0; continue; }
        // not written yet, or enough aggregates remembered: wait for this record
        if (++polls > p.spin_cap) {
            atomicExch(p.header + 2, rlcs::kDeviceTimeout);
            return 0.f;
        }
        __nanosleep(64);
    }
    for (int i = n - 1; i >= 0; --i) start = fmaf(sb[i], start, sa[i]);
    return start;
}

template <int ALGO, bool TRUNC, int W, int C>
__global__ void __launch_bounds__(32 * W) tm_block_chained_kernel(const TmParams p_in) {
    constexpr bool FWD = tm_forward(ALGO);
    constexpr bool ONE_WALK = tm_row_mask(ALGO);             // vector traces: one flag per timestep
    __shared__ unsigned s_ticket;
    __shared__ float s_carry[32 * C];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    if (threadIdx.x == 0) s_ticket = atomicAdd(p_in.header + 63, 1u);
    __syncthreads();
    const unsigned chains = p_in.colblocks * (unsigned)p_in.batch;
    const unsigned ks = s_ticket / chains;                   // chunk in scan order
    const unsigned chain = s_ticket - ks * chains;
    const unsigned z = chain / p_in.colblocks;
    const unsigned xb = chain - z * p_in.colblocks;
    if (ks >= p_in.chunks) return;
    const TmParams p = batch_slice<ALGO>(p_in, z);
    const unsigned k = FWD ? ks : p.chunks - 1 - ks;
    const long long n0 = (long long)xb * (32 * C);
    const bool write = n0 + C * lane < p.N;
    const unsigned t_lo = k * p.chunk, t_hi = min(p.T, t_lo + p.chunk), len = t_hi - t_lo;
    // Steps the incoming carry reaches: those before the chunk's first cut (the carry into step t is
    // cut iff dones[t-1]; chunk 0 takes no carry).  Every warp finds the bound for itself.
    unsigned qdefer = 0;
    if constexpr (ONE_WALK) {
        if (ks > 0) {
            qdefer = len;
            for (unsigned q0 = 0; q0 < len; q0 += 32) {
                const unsigned q = q0 + lane;
                const bool cut = q < len && __ldg(p.dones + t_lo + q - 1) != 0;
                const unsigned m = __ballot_sync(0xffffffffu, cut);
                if (m != 0) { qdefer = q0 + (unsigned)__ffs((int)m) - 1; break; }
            }
        }
    }
    float A[C], P[C];
#pragma unroll
    for (int c = 0; c < C; ++c) A[c] = 0.f;
    block_walk<ALGO, TRUNC, ONE_WALK ? 3 : 1, W, C>(p, n0, k, A, P, qdefer);
    if (w == 0) {
        const long long rec0 = (long long)z * p.chunks * p.npad + n0 + C * lane;
#pragma unroll
        for (int c = 0; c < C; ++c) {
            float carry = 0.f;
            if (write && (long long)s_ticket != p.mute_ticket) {
                uint4* mine = p.records + rec0 + c + (long long)ks * p.npad;
                rlcs::st_volatile_u4(mine, make_uint4(__float_as_uint(A[c]), 1u, __float_as_uint(P[c]), 1u));
                if (ks > 0) carry = chained_carry(p, rec0 + c, ks);
                if (ks + 1 < p.chunks)
                    rlcs::st_volatile_u4(mine, make_uint4(__float_as_uint(fmaf(P[c], carry, A[c])), 2u, 0u, 2u));
            }
            s_carry[C * lane + c] = carry;
        }
    }
    __syncthreads();                                         // the carries are there, and every warp is done with the walk
    if constexpr (!ONE_WALK) {
#pragma unroll
        for (int c = 0; c < C; ++c) A[c] = s_carry[C * lane + c];
        block_walk<ALGO, TRUNC, 2, W, C>(p, n0, k, A, P);
    } else {
        // Finish the deferred steps: value from carry 0 (ring, f0 entry) + sensitivity * carry.  Rows go
        // round-robin over the warps.  With the shared decay the sensitivity of step q is decay^(q+1).
        if (qdefer == 0 || !write) return;
        using SV = StageView<ALGO, TRUNC, W, C>;
        extern __shared__ __align__(16) unsigned char tm_smem[];
        constexpr int R = SV::KR * W;
        constexpr int fstage = R * SV::NF * 128 * C;
        float c0[C];
#pragma unroll
        for (int c = 0; c < C; ++c) c0[c] = s_carry[C * lane + c];
        float pw = p.decay, step = 1.f;                      // decay^(w+1), decay^W
        if constexpr (!tm_vec_beta(ALGO)) {
            for (int x = 0; x < w; ++x) pw *= p.decay;
            for (int x = 0; x < W; ++x) step *= p.decay;
        }
        float* dst = p.out0 + (long long)t_lo * p.N + n0 + C * lane;
        for (unsigned q = w; q < qdefer; q += W) {
            const SV sv{tm_smem + (q / R) * fstage, nullptr};
            float v[C], sens[C];
            lds_f<C>(sv.f(0, q % R), lane, v);
            if constexpr (tm_vec_beta(ALGO)) lds_f<C>(sv.f(1, q % R), lane, sens);
#pragma unroll
            for (int c = 0; c < C; ++c) v[c] = fmaf(tm_vec_beta(ALGO) ? sens[c] : pw, c0[c], v[c]);
            stg_f<C>(dst + (long long)q * p.N, v);
            pw *= step;
        }
    }
}

// Chain an environment's chunks in scan order: carry into chunk k = a_j + b_j * (carry into j) for the
// scan-order predecessor j.  Overwrites agg_a[k] with the carry into chunk k.
template <bool FWD>
__global__ void __launch_bounds__(kThreads) tm_chain_kernel(const TmParams p) {
    const long long n = (long long)blockIdx.x * kThreads + threadIdx.x;
    if (n >= p.N) return;
    float carry = 0.f;
    for (unsigned s = 0; s < p.chunks; ++s) {
        const unsigned k = FWD ? s : p.chunks - 1 - s;
        const long long i = (long long)k * p.N + n;
        const float a = p.agg_a[i], b = p.agg_b[i];
        p.agg_a[i] = carry;
        carry = fmaf(b, carry, a);
    }
}

// ---------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------

// SM count and shared memory per SM of the current device (usable by thread blocks; each resident
// block also costs 1 KB), see rlcs_device.cuh
inline long long sm_count() { return rlcs_device::limits().sms; }
inline long long smem_per_sm() { return (long long)rlcs_device::limits().smem_per_sm; }

// How the time axis is cut.  Depends on N and T only, so that the workspace size does.
void plan_chunks(long long N, long long T, unsigned* chunk, unsigned* chunks) {
    // A thread block owns 32 columns.  From about two blocks for every three SMs upward whole columns
    // are walked; with fewer the time axis is cut.  A cut costs a second read of the inputs whatever
    // the number of chunks, so chunks are short (two blocks per SM in total), but not below 64 steps.
    *chunk = (unsigned)T;
    *chunks = 1;
    const long long groups = (N + 31) / 32;
    if (groups >= 96) return;
    const long long k = (2 * sm_count() + groups - 1) / groups;
    long long len = (T + k - 1) / k;
    if (len < 64) len = 64;
    len = (len + kRows - 1) / kRows * kRows;
    if (len >= T) return;
    *chunk = (unsigned)len;
    *chunks = (unsigned)((T + len - 1) / len);
}

// Columns per lane, warps per block and ring depth for tm_block_kernel.  Two columns per lane when
// that still leaves two blocks per SM (and the outputs allow 8-byte stores); sixteen or eight warps when blocks
// are scarce (fewer than one or two per SM), else four.  The kernel is bound by issue slots and dependent-ALU latency as much as by
// HBM, so resident warps come first: the ring is as deep as still lets min(blocks per SM, 6) blocks
// share an SM, no deeper than keeps about 16 MB in flight over the grid, and at least 3.
size_t plan_block(TmParams& p, int rows, int row_bytes, bool trunc, bool wide_ok, bool whole_chunk = false) {
    int C = 1;
    const long long batch = p.batch > 0 ? p.batch : 1;
    if (wide_ok && (p.N + 63) / 64 * p.chunks * batch >= 2 * sm_count()) C = 2;
    const long long blocks = (p.N + 32 * C - 1) / (32 * C) * p.chunks * batch;
    const long long sms = sm_count(), smem = smem_per_sm();
    int W = C == 2 ? 4 : blocks < sms ? 16 : blocks < 2 * sms ? 8 : 4;
    long long stage, mstage, fixed;
    auto size = [&]() {
        stage = (long long)rows * W * row_bytes * C;
        mstage = (long long)rows * W * (trunc ? 64 : 32) * C;
        fixed = 2 * mstage + (W * 512 + 512) * C;               // mask ring's two extra slots, aggregates, edges
    };
    auto block_bytes = [&](long long S) { return S * stage + fixed; };
    size();
    while (W > 4 && block_bytes(3) + 1024 > smem) { W /= 2; size(); }   // the minimum ring must fit
    long long resident = (blocks + sms - 1) / sms;
    if (resident > 6) resident = 6;
    while (resident > 1 && resident * (block_bytes(3) + 1024) > smem) --resident;
    long long S = 2 + ((16ll << 20) + blocks * stage - 1) / (blocks * stage);
    const long long nst = ((long long)p.chunk + rows * W - 1) / (rows * W);
    if (S > nst + 1) S = nst + 1;
    if (S > kMaxStages) S = kMaxStages;
    while (S > 3 && resident * (block_bytes(S) + 1024) > smem) --S;
    if (S < 3) S = 3;
    // the chained kernel of the vector traces keeps its chunk (about 32 KB) in the ring: the entries of
    // the steps before the first cut are reused after the walk
    if (whole_chunk && p.records != nullptr && S < nst) S = nst;
    p.stages = (int)S;
    p.warps_per_block = W;
    p.cols_per_lane = C;
    return (size_t)block_bytes(S);
}

int g_force_cols = 0;    // test hook: 1 = one column per lane whatever the size

inline bool aligned8(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 7u) == 0; }

template <typename K>
bool allow_smem(K kernel, size_t bytes) {
    if (bytes <= 48 * 1024) return true;
    return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(smem_per_sm() - 1024)) == cudaSuccess;
}

// Chunks of the chained kernel: about 32 KB of inputs per block and chunk.  The vector traces keep
// the chunk in the ring while it is walked once (measured at 64 x 16384 x 64 / 16 x 65536 x 64 with a
// decay tensor, fraction of the copy bandwidth: 16 KB 0.65 / 0.60, 32 KB 0.67 / 0.69, 64 KB 0.59 /
// 0.58); the time-major entry points walk it twice, and the chunks of all resident blocks stay in L2
// in between.  A multiple of 64 steps (every stage size divides it), at least 64.
constexpr unsigned kChainedMinChunk = 64;
unsigned chained_chunk_len(int row_bytes) {
    unsigned len = (32768u / (unsigned)row_bytes) / 64u * 64u;
    return len < kChainedMinChunk ? kChainedMinChunk : len;
}
// bytes of workspace that cover the records of any algorithm's chunking, plus the header
size_t chained_ws_bytes(long long N, long long T, long long batch) {
    const long long npad = (N + 63) / 64 * 64;
    const long long chunks = (T + kChainedMinChunk - 1) / kChainedMinChunk;
    return 256 + sizeof(uint4) * (size_t)(npad * chunks * batch);
}

int g_force_chained = 0;   // test hook: 1 = never the chained kernel, 2 = the chained kernel whenever T allows a cut

template <int ALGO, bool TRUNC, int W, int C>
int launch_block(const TmParams& p_in, size_t smem, cudaStream_t s) {
    TmParams p = p_in;
    const unsigned colblocks = (unsigned)((p.N + 32 * C - 1) / (32 * C));
    const long long batch = p.batch > 0 ? p.batch : 1;
    if (p.chunks > 1 && p.records != nullptr) {
        p.colblocks = colblocks;
        p.npad = (long long)colblocks * 32 * C;
        p.batch = batch;
        const long long blocks = (long long)colblocks * batch * p.chunks;
        if (blocks > 0x7fffffffll) return RLCS_ERR_SIZE;
        auto kernel = tm_block_chained_kernel<ALGO, TRUNC, W, C>;
        if (!allow_smem(kernel, smem)) return RLCS_ERR_CUDA;
        // the ticket counter (the header's last word) and the records behind it
        const size_t clear = 4 + sizeof(uint4) * (size_t)(p.npad * p.chunks * batch);
        if (cudaMemsetAsync(reinterpret_cast<unsigned char*>(p.header) + 252, 0, clear, s) != cudaSuccess) return RLCS_ERR_CUDA;
        kernel<<<(unsigned)blocks, 32 * W, smem, s>>>(p);
        return cudaGetLastError() == cudaSuccess ? RLCS_OK : RLCS_ERR_CUDA;
    }
    const dim3 grid(colblocks, p.chunks, (unsigned)batch);
    if (p.chunks == 1) {
        if (!allow_smem(tm_block_kernel<ALGO, TRUNC, 0, W, C>, smem)) return RLCS_ERR_CUDA;
        // the uncut walk is launched like the row-major scan kernels (see launch_scan in rlcs_launch.cuh)
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = grid;
        cfg.blockDim = dim3(32 * W, 1, 1);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = s;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = rlcs_hooks::g_pdl ? 1 : 0;
        return cudaLaunchKernelEx(&cfg, tm_block_kernel<ALGO, TRUNC, 0, W, C>, p) == cudaSuccess ? RLCS_OK : RLCS_ERR_CUDA;
    } else {
        if (!allow_smem(tm_block_kernel<ALGO, TRUNC, 1, W, C>, smem) || !allow_smem(tm_block_kernel<ALGO, TRUNC, 2, W, C>, smem))
            return RLCS_ERR_CUDA;
        tm_block_kernel<ALGO, TRUNC, 1, W, C><<<grid, 32 * W, smem, s>>>(p);
        tm_chain_kernel<tm_forward(ALGO)><<<(unsigned)((p.N + kThreads - 1) / kThreads), kThreads, 0, s>>>(p);
        tm_block_kernel<ALGO, TRUNC, 2, W, C><<<grid, 32 * W, smem, s>>>(p);
    }
    return cudaGetLastError() == cudaSuccess ? RLCS_OK : RLCS_ERR_CUDA;
}

template <int ALGO, bool TRUNC>
int launch(TmParams p, bool staged, cudaStream_t s) {
    constexpr bool FWD = tm_forward(ALGO);
    const unsigned gx_chain = (unsigned)((p.N + kThreads - 1) / kThreads);
    if (staged) {
        // Two columns per lane pay where registers allow it (measured: GAE and TD(lambda) without
        // truncation handling, +4 %; with it, or with three or four float inputs, 128-168 registers
        // per thread cost more occupancy than the shared addressing saves).
        constexpr bool kWide = !TRUNC && (ALGO == kGae || ALGO == kTdLambda);
        const bool wide_ok = kWide && g_force_cols != 1 && aligned8(p.out0) && aligned8(p.out1);
        if (p.header != nullptr && g_force_chained != 1 && (p.chunks > 1 || g_force_chained == 2)) {
            // the time axis is cut: one launch with chained carries instead of three with a second read
            const unsigned len = chained_chunk_len(tm_row_bytes(ALGO, TRUNC));
            if (len < p.T) {
                p.chunk = len;
                p.chunks = (p.T + len - 1) / len;
                p.records = reinterpret_cast<uint4*>(reinterpret_cast<unsigned char*>(p.header) + 256);
            }
        }
        const size_t smem = plan_block(p, tm_rows(ALGO), tm_row_bytes(ALGO, TRUNC), TRUNC, wide_ok);
        if constexpr (kWide) {
            if (p.cols_per_lane == 2) return launch_block<ALGO, TRUNC, 4, 2>(p, smem, s);
        }
        if (p.warps_per_block == 16) return launch_block<ALGO, TRUNC, 16, 1>(p, smem, s);
        return p.warps_per_block == 8 ? launch_block<ALGO, TRUNC, 8, 1>(p, smem, s) : launch_block<ALGO, TRUNC, 4, 1>(p, smem, s);
    } else {
        const dim3 grid(gx_chain, p.chunks);
        if (p.chunks == 1) {
            tm_kernel<ALGO, TRUNC, 0><<<grid, kThreads, 0, s>>>(p);
        } else {
            tm_kernel<ALGO, TRUNC, 1><<<grid, kThreads, 0, s>>>(p);
            tm_chain_kernel<FWD><<<gx_chain, kThreads, 0, s>>>(p);
            tm_kernel<ALGO, TRUNC, 2><<<grid, kThreads, 0, s>>>(p);
        }
    }
    return cudaGetLastError() == cudaSuccess ? RLCS_OK : RLCS_ERR_CUDA;
}

inline bool aligned4(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 3u) == 0; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

constexpr unsigned kDefaultSpinCap = 1u << 22;    // polls of one record (64 ns apart or more) before a chained kernel gives up
unsigned spin_cap() { return rlcs_hooks::g_spin_cap > 0 ? (unsigned)rlcs_hooks::g_spin_cap : kDefaultSpinCap; }

// workspace of the time-major entry points: 256-byte header, then whichever is larger of the chained
// kernel's records and the three-launch path's two aggregate arrays
size_t tm_ws_bytes(long long N, long long T, unsigned chunks) {
    const size_t chained = chained_ws_bytes(N, T, 1);
    const size_t three = 256 + 2 * sizeof(float) * (size_t)N * chunks;
    return chained > three ? chained : three;
}
inline bool unit(float v) { return v >= 0.f && v <= 1.f; }

// the staged kernels copy 16-byte pieces of every per-step input
bool can_stage(const TmParams& p) {
    // (the ring kernels step from row to row with a 32-bit byte offset)
    if (p.N % 16 != 0 || p.N > (1ll << 28)) return false;
    const void* in[] = {p.f0, p.f1, p.f2, p.f3, p.dones, p.truncs};
    for (const void* q : in)
        if (q != nullptr && !aligned16(q)) return false;
    return true;
}

int g_force_path = 0;   // test hook: 1 = register path only, 2 = staged wherever alignment allows (the default)

// shared validation and workspace wiring; returns RLCS_OK with *skip = true for empty problems
int prepare(TmParams& p, int64_t N, int64_t T, const void* const* f32, int nf32, const uint8_t* dones,
            const uint8_t* truncs, const float* trunc_bootstrap, bool backward, void* workspace, size_t workspace_bytes,
            bool* skip) {
    *skip = false;
    if (N < 0 || T < 0 || T > (int64_t(1) << 31) - 1) return RLCS_ERR_SIZE;
    if (N == 0 || T == 0) { *skip = true; return RLCS_OK; }
    if (N > (int64_t(1) << 40) / T) return RLCS_ERR_SIZE;
    if (dones == nullptr) return RLCS_ERR_NULL;
    if (backward && (truncs == nullptr) != (trunc_bootstrap == nullptr)) return RLCS_ERR_NULL;
    for (int i = 0; i < nf32; ++i)
        if (f32[i] != nullptr && !aligned4(f32[i])) return RLCS_ERR_ALIGN;
    p.N = N;
    p.T = (unsigned)T;
    plan_chunks(N, T, &p.chunk, &p.chunks);
    p.spin_cap = spin_cap();
    p.mute_ticket = rlcs_hooks::g_mute_tile;
    if (p.chunks > 1 || g_force_chained == 2) {
        const size_t need = tm_ws_bytes(N, T, p.chunks);
        if (workspace == nullptr || workspace_bytes < need) return RLCS_ERR_WORKSPACE;
        if (!aligned16(workspace)) return RLCS_ERR_ALIGN;
        // header (256 bytes), then either the chained kernel's records or the three-launch path's aggregates
        p.header = static_cast<unsigned*>(workspace);
        p.agg_a = reinterpret_cast<float*>(static_cast<unsigned char*>(workspace) + 256);
        p.agg_b = p.agg_a + (size_t)N * p.chunks;
    }
    return RLCS_OK;
}

template <int ALGO, bool TRUNC>
int run(const TmParams& p, void* cuda_stream) {
    const bool staged = g_force_path != 1 && can_stage(p);
    return launch<ALGO, TRUNC>(p, staged, static_cast<cudaStream_t>(cuda_stream));
}

}  // namespace

// Vector-valued eligibility traces for few long rows (called from rlcs_elig_vec.cu, today for the
// per-component decay only): every row n is a time-major [T, D] problem with one flag per timestep;
// one thread block per 32 components and row streams the row once through the shared-memory ring,
// its warps splitting every stage in time.
namespace rlcs_internal {

// usable when every row of D floats can be copied in 16-byte pieces and there are enough blocks
// Few long rows: the time axis is cut and the chunks chained inside one launch.  Measured at D = 64
// (fraction of the copy bandwidth, uncut -> chained): shared decay 0.49 -> 0.59 with 128 blocks,
// 0.56 -> 0.59 with 256, 0.58 -> 0.59 with 512, 0.81 -> 0.59 with 1024; per-component decay 0.67 ->
// 0.59 with 128 blocks, 0.75 -> 0.59 with 256.  So the shared decay cuts below four blocks per SM, the
// per-component decay only where rows and components alone give too few blocks to run uncut at all
// (fewer than 96).  (More warps per block than plan_block gives lose with either decay; fewer lose
// below two blocks per SM.)
bool vec_trace_block_cuts(int64_t N, int64_t T, int64_t D, bool perdim) {
    if (g_force_chained == 1) return false;
    const unsigned len = chained_chunk_len(tm_row_bytes(perdim ? kTmVecBeta : kTmVec, false));
    if ((int64_t)len >= T) return false;
    return g_force_chained == 2 || (D + 31) / 32 * N < (perdim ? 96 : 4 * sm_count());
}

// shapes the block kernel takes: rows of D floats copied in 16-byte pieces, and enough blocks -- from
// rows and components alone, or from the chunks of a cut time axis
bool vec_trace_block_shape_ok(int64_t N, int64_t T, int64_t D, bool perdim) {
    if (g_force_path == 1) return false;
    if (D % 4 != 0 || D < 32 || D > (1ll << 28) || T < 64 || N > 65535) return false;
    return (D + 31) / 32 * N >= 96 || vec_trace_block_cuts(N, T, D, perdim);
}
bool vec_trace_block_usable(const float* x, const float* beta, int64_t N, int64_t T, int64_t D) {
    return vec_trace_block_shape_ok(N, T, D, beta != nullptr) && aligned16(x) && (beta == nullptr || aligned16(beta));
}

// header plus one record per row, chunk and (padded) component; the vector kernels use one column per lane
size_t vec_chained_ws_bytes(int64_t N, int64_t T, int64_t D, bool perdim) {
    const long long len = chained_chunk_len(tm_row_bytes(perdim ? kTmVecBeta : kTmVec, false));
    const long long npad = (D + 31) / 32 * 32, chunks = (T + len - 1) / len;
    return 256 + sizeof(uint4) * (size_t)(npad * chunks * N);
}

size_t vec_trace_block_workspace_bytes(int64_t N, int64_t T, int64_t D, bool perdim) {
    return vec_trace_block_shape_ok(N, T, D, perdim) && vec_trace_block_cuts(N, T, D, perdim) ? vec_chained_ws_bytes(N, T, D, perdim) : 0;
}

int vec_trace_block(const float* x, const float* beta, const uint8_t* dones, float* traces, int64_t N, int64_t T, int64_t D,
                    float decay, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    TmParams p = {};
    p.f0 = x; p.f1 = beta; p.dones = dones; p.out0 = traces;
    p.N = D; p.T = (unsigned)T; p.chunk = (unsigned)T; p.chunks = 1;
    p.decay = decay;
    p.batch = N; p.batch_stride = T * D;
    p.spin_cap = spin_cap();
    p.mute_ticket = rlcs_hooks::g_mute_tile;
    const bool perdim = beta != nullptr;
    if (vec_trace_block_cuts(N, T, D, perdim)) {
        if (workspace == nullptr || workspace_bytes < vec_chained_ws_bytes(N, T, D, perdim)) return RLCS_ERR_WORKSPACE;
        if (!aligned16(workspace)) return RLCS_ERR_ALIGN;
        p.header = static_cast<unsigned*>(workspace);
        p.records = reinterpret_cast<uint4*>(static_cast<unsigned char*>(workspace) + 256);
        p.chunk = chained_chunk_len(tm_row_bytes(perdim ? kTmVecBeta : kTmVec, false));
        p.chunks = (p.T + p.chunk - 1) / p.chunk;
    }
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    auto go = [&](auto algo_tag) {
        constexpr int ALGO = decltype(algo_tag)::value;
        const size_t smem = plan_block(p, tm_rows(ALGO), tm_row_bytes(ALGO, false), false, false, true);
        if (p.warps_per_block == 16) return launch_block<ALGO, false, 16, 1>(p, smem, s);
        if (p.warps_per_block == 8) return launch_block<ALGO, false, 8, 1>(p, smem, s);
        return launch_block<ALGO, false, 4, 1>(p, smem, s);
    };
    if (!perdim) return go(std::integral_constant<int, kTmVec>{});
    // deeper stages while every block is resident at once (up to ten 128-thread blocks per SM)
    const long long blocks = (D + 31) / 32 * N * p.chunks;
    return (p.chunks == 1 && blocks < 10 * sm_count()) ? go(std::integral_constant<int, kTmVecBeta16>{})
                                                 : go(std::integral_constant<int, kTmVecBeta>{});
}

}  // namespace rlcs_internal

extern "C" {

size_t rlcs_time_major_workspace_bytes(int64_t N, int64_t T) {
    if (N <= 0 || T <= 0 || T > (int64_t(1) << 31) - 1) return 0;
    unsigned chunk, chunks;
    plan_chunks(N, T, &chunk, &chunks);
    return (chunks > 1 || g_force_chained == 2) ? tm_ws_bytes(N, T, chunks) : 0;
}

void rlcs_debug_time_major_path(int path) {
    g_force_path = path == 1 ? 1 : 0;
    g_force_cols = path == 3 ? 1 : 0;
    g_force_chained = path == 4 ? 1 : path == 5 ? 2 : 0;
}

int rlcs_gae_time_major(const float* rewards, const float* values, const uint8_t* dones, const uint8_t* truncs,
                        const float* trunc_bootstrap, const float* bootstrap, float* advantages, float* returns,
                        int64_t N, int64_t T, float gamma, float lambda, void* workspace, size_t workspace_bytes,
                        void* cuda_stream) {
    if (!unit(gamma) || !unit(lambda)) return RLCS_ERR_ARG;
    TmParams p = {};
    bool skip;
    const void* f[] = {rewards, values, trunc_bootstrap, bootstrap, advantages, returns};
    int st = prepare(p, N, T, f, 6, dones, truncs, trunc_bootstrap, true, workspace, workspace_bytes, &skip);
    if (st != RLCS_OK || skip) return st;
    if (!rewards || !values || !advantages) return RLCS_ERR_NULL;
    p.f0 = rewards; p.f1 = values; p.dones = dones; p.truncs = truncs; p.trunc_boot = trunc_bootstrap; p.boot = bootstrap;
    p.out0 = advantages; p.out1 = returns; p.gamma = gamma; p.decay = gamma * lambda;
    return truncs ? run<kGae, true>(p, cuda_stream) : run<kGae, false>(p, cuda_stream);
}

int rlcs_vtrace_time_major(const float* rewards, const float* values, const float* log_rhos, const uint8_t* dones,
                           const uint8_t* truncs, const float* trunc_bootstrap, const float* bootstrap, float* vs,
                           float* pg_advantages, int64_t N, int64_t T, float gamma, float rho_bar, float c_bar,
                           void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (!unit(gamma) || !(rho_bar >= 0.f) || !(c_bar >= 0.f)) return RLCS_ERR_ARG;
    TmParams p = {};
    bool skip;
    const void* f[] = {rewards, values, log_rhos, trunc_bootstrap, bootstrap, vs, pg_advantages};
    int st = prepare(p, N, T, f, 7, dones, truncs, trunc_bootstrap, true, workspace, workspace_bytes, &skip);
    if (st != RLCS_OK || skip) return st;
    if (!rewards || !values || !log_rhos || !vs) return RLCS_ERR_NULL;
    p.f0 = rewards; p.f1 = values; p.f3 = log_rhos; p.dones = dones; p.truncs = truncs; p.trunc_boot = trunc_bootstrap;
    p.boot = bootstrap; p.out0 = vs; p.out1 = pg_advantages; p.gamma = gamma; p.rho_bar = rho_bar; p.c_bar = c_bar;
    return truncs ? run<kVtrace, true>(p, cuda_stream) : run<kVtrace, false>(p, cuda_stream);
}

int rlcs_retrace_time_major(const float* rewards, const float* q_sa, const float* expected_q, const float* log_rhos,
                            const uint8_t* dones, const uint8_t* truncs, const float* trunc_bootstrap,
                            const float* bootstrap, float* q_targets, int64_t N, int64_t T, float gamma, float lambda,
                            float c_bar, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (!unit(gamma) || !unit(lambda) || !(c_bar >= 0.f)) return RLCS_ERR_ARG;
    TmParams p = {};
    bool skip;
    const void* f[] = {rewards, q_sa, expected_q, log_rhos, trunc_bootstrap, bootstrap, q_targets};
    int st = prepare(p, N, T, f, 7, dones, truncs, trunc_bootstrap, true, workspace, workspace_bytes, &skip);
    if (st != RLCS_OK || skip) return st;
    if (!rewards || !q_sa || !expected_q || !log_rhos || !q_targets) return RLCS_ERR_NULL;
    p.f0 = rewards; p.f1 = q_sa; p.f2 = expected_q; p.f3 = log_rhos; p.dones = dones; p.truncs = truncs;
    p.trunc_boot = trunc_bootstrap; p.boot = bootstrap; p.out0 = q_targets; p.gamma = gamma; p.aux = gamma * lambda;
    p.c_bar = c_bar;
    return truncs ? run<kRetrace, true>(p, cuda_stream) : run<kRetrace, false>(p, cuda_stream);
}

int rlcs_td_lambda_time_major(const float* rewards, const float* values, const uint8_t* dones, const uint8_t* truncs,
                              const float* trunc_bootstrap, const float* bootstrap, float* returns, int64_t N,
                              int64_t T, float gamma, float lambda, void* workspace, size_t workspace_bytes,
                              void* cuda_stream) {
    if (!unit(gamma) || !unit(lambda)) return RLCS_ERR_ARG;
    TmParams p = {};
    bool skip;
    const void* f[] = {rewards, values, trunc_bootstrap, bootstrap, returns};
    int st = prepare(p, N, T, f, 5, dones, truncs, trunc_bootstrap, true, workspace, workspace_bytes, &skip);
    if (st != RLCS_OK || skip) return st;
    if (!rewards || !values || !returns) return RLCS_ERR_NULL;
    p.f0 = rewards; p.f1 = values; p.dones = dones; p.truncs = truncs; p.trunc_boot = trunc_bootstrap; p.boot = bootstrap;
    p.out0 = returns; p.gamma = gamma; p.decay = gamma * lambda; p.aux = gamma * (1.f - lambda);
    return truncs ? run<kTdLambda, true>(p, cuda_stream) : run<kTdLambda, false>(p, cuda_stream);
}

int rlcs_discounted_return_time_major(const float* rewards, const uint8_t* dones, const uint8_t* truncs,
                                      const float* trunc_bootstrap, const float* bootstrap, float* returns, int64_t N,
                                      int64_t T, float gamma, void* workspace, size_t workspace_bytes,
                                      void* cuda_stream) {
    if (!unit(gamma)) return RLCS_ERR_ARG;
    TmParams p = {};
    bool skip;
    const void* f[] = {rewards, trunc_bootstrap, bootstrap, returns};
    int st = prepare(p, N, T, f, 4, dones, truncs, trunc_bootstrap, true, workspace, workspace_bytes, &skip);
    if (st != RLCS_OK || skip) return st;
    if (!rewards || !returns) return RLCS_ERR_NULL;
    p.f0 = rewards; p.dones = dones; p.truncs = truncs; p.trunc_boot = trunc_bootstrap; p.boot = bootstrap;
    p.out0 = returns; p.gamma = gamma; p.decay = gamma;
    return truncs ? run<kDisc, true>(p, cuda_stream) : run<kDisc, false>(p, cuda_stream);
}

int rlcs_elig_trace_time_major(const float* x, const uint8_t* dones, float* traces, int64_t N, int64_t T, float gamma,
                               float lambda, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (!unit(gamma) || !unit(lambda)) return RLCS_ERR_ARG;
    TmParams p = {};
    bool skip;
    const void* f[] = {x, traces};
    int st = prepare(p, N, T, f, 2, dones, nullptr, nullptr, false, workspace, workspace_bytes, &skip);
    if (st != RLCS_OK || skip) return st;
    if (!x || !traces) return RLCS_ERR_NULL;
    p.f0 = x; p.dones = dones; p.out0 = traces; p.decay = gamma * lambda;
    return run<kElig, false>(p, cuda_stream);
}

int rlcs_episodic_prefix_sum_time_major(const float* x, const uint8_t* dones, float* sums, int64_t N, int64_t T,
                                        int starts_at, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    TmParams p = {};
    bool skip;
    const void* f[] = {x, sums};
    int st = prepare(p, N, T, f, 2, dones, nullptr, nullptr, false, workspace, workspace_bytes, &skip);
    if (st != RLCS_OK || skip) return st;
    if (!x || !sums) return RLCS_ERR_NULL;
    p.f0 = x; p.dones = dones; p.out0 = sums; p.decay = 1.f; p.starts_at = starts_at != 0;
    return run<kPrefix, false>(p, cuda_stream);
}

}  // extern "C"
