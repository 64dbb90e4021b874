/*
 * rlcs -- fused credit-assignment scans for reinforcement learning on NVIDIA B200 (sm_100a).
 *
 * Seven entry points, one fused kernel launch each.  Every call reads raw rollout tensors of
 * shape [N, T] (N = num_envs rows, T = timesteps per row), builds the per-step affine
 * coefficients (alpha_t, beta_t) of Table 1 on chip, and solves the first-order linear recurrence
 * of Eq. 1,  A_t = alpha_t + beta_t * A_{t+1}  (or the forward mirror with A_{t-1}),  as a
 * segmented associative scan under the combine operator of Eq. 2.  Episode boundaries reset the
 * scan; bootstrap values enter at truncations and at the rollout-window edge (Section 3.2).
 *
 * CONVENTIONS COMMON TO ALL ENTRY POINTS
 *
 * Pointers.  Every pointer except `cuda_stream` is a DEVICE pointer.  The caller owns every
 *   buffer, including `workspace`; the library allocates nothing and keeps no state between
 *   calls (apart from a per-device cache of launch configurations).  Outputs must not overlap
 *   inputs or each other.
 * Layout.  Every [N, T] tensor is contiguous row-major: element (n, t) at index n*T + t.
 *   Floating-point tensors are fp32 (Section 4.4: the method is fp32-only).  Masks are uint8,
 *   zero = false, any non-zero value = true.
 * Flags.  For the five backward algorithms `dones` is the termination flag d^term and `truncs`
 *   the truncation flag d^trunc; d_t = d^term_t OR d^trunc_t severs the recurrence (Table 1
 *   caption).  `truncs` and `trunc_bootstrap` are both NULL (no per-step truncation handling,
 *   the HAS_TRUNCATIONS=False case of Section 4.2) or both non-NULL.  The two forward scans take
 *   ONE already-combined flag (term OR trunc) in `dones`.
 * Successor value of step t (Section 3.2), written X_next(t) below, for X = values or expected_q:
 *     0                       if dones[n,t]            (termination wins when both flags are set)
 *     trunc_bootstrap[n,t]    else if truncs[n,t]      (supplied continuation value)
 *     bootstrap[n]            else if t == T-1         (rollout-window edge; NULL pointer = 0,
 *                                                       the HAS_BOOTSTRAP=False case)
 *     X[n,t+1]                otherwise.
 *   The recurrence continues from t into t+1 ("cont_t") only when no flag is set at t and
 *   t < T-1.  trunc_bootstrap is read only where truncs is set and dones is not.
 * Sizes.  N >= 0, 0 <= T < 2^31, N*T < 2^40.  N == 0 or T == 0 returns RLCS_OK without a launch.
 * Parameters.  gamma and lambda must lie in [0, 1] (1 is valid); clip thresholds must be >= 0
 *   (+inf = no clipping).  NaN is rejected.
 * Alignment.  fp32 pointers must be 4-byte aligned.  When every fp32 pointer is 32-byte aligned
 *   and every mask pointer 16-byte aligned the vectorised kernels run (256-bit accesses, bulk
 *   copies); otherwise a slower element-wise variant of the same kernel is used (same results).
 * Workspace.  The kernels cut the flattened [N*T] array into tiles of 512 to 2048 steps, one per
 *   thread block.  When T divides the tile, or a whole number of rows nearly fills it (at least 70 %,
 *   with every thread still holding a whole chunk: T = 1000, 2000, 500, 250, 200, 100, ...), tiles
 *   are aligned to rows and blocks are independent.  Otherwise rows straddle tiles and need a carry
 *   between thread blocks, passed
 *   through `workspace`: at least rlcs_workspace_bytes(N, T) bytes, 16-byte aligned, initialised
 *   once with rlcs_workspace_init and then reusable by any number of calls, of any of the entry
 *   points, that are ordered on one stream.  Two calls that may run concurrently need two
 *   workspaces.  When rlcs_workspace_bytes(N, T) is 0 the workspace may be NULL.
 * Execution.  Work is enqueued on `cuda_stream` (a cudaStream_t passed as void*; NULL = the
 *   default stream) and the call returns without synchronising.  The row-major scan kernels, the
 *   follow-up kernels of rlcs_gae_normalized and the time-major ring kernel (uncut time axis) are
 *   launched with programmatic stream serialisation: their thread blocks may be placed on the GPU
 *   while the preceding kernel of the stream drains, but they wait for that kernel's completion
 *   (and the visibility of its writes) before their first access to global memory -- caller
 *   tensors and workspace alike -- so the stream's ordering guarantees are unchanged.  Argument
 *   errors are returned before anything is launched.  The only device-side wait is the bounded
 *   carry wait between thread blocks.  A block only ever waits for tiles that precede its own in
 *   scan order, and tiles are assigned by launch index: the look-back relies on the hardware
 *   starting thread blocks in index order, as every current GPU does but CUDA does not promise.
 *   Should a block ever wait for one that has not been started, nothing hangs: the wait runs out
 *   of polls, the kernel still terminates normally, the outputs of that call are unspecified, and rlcs_last_device_status reports RLCS_ERR_TIMEOUT.
 * Inputs must be finite.  A reset is a decay of exactly 0 inside the scan (0 * finite severs
 *   exactly); successor values at resets are selected, never multiplied.  A NaN or infinity in one
 *   episode can therefore reach the flagged last step of the preceding episode, but nothing else.
 * Results are deterministic: the same inputs give bit-identical outputs on every call.
 */
#ifndef RLCS_H_
#define RLCS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    RLCS_OK = 0,
    RLCS_ERR_NULL = 1,       /* a required pointer is NULL, or exactly one of truncs/trunc_bootstrap */
    RLCS_ERR_SIZE = 2,       /* negative or too large N / T */
    RLCS_ERR_ARG = 3,        /* gamma / lambda / clip out of range or NaN */
    RLCS_ERR_ALIGN = 4,      /* fp32 pointer not 4-byte aligned, workspace not 16-byte aligned */
    RLCS_ERR_WORKSPACE = 5,  /* workspace NULL or too small for this (N, T) */
    RLCS_ERR_CUDA = 6,       /* the launch itself failed (cudaGetLastError) */
    RLCS_ERR_TIMEOUT = 7,    /* device status: a bounded carry wait gave up */
    RLCS_ERR_LIMIT = 8,      /* rlcs_gae_no_alloc: the problem needs more scratch than the built-in array holds */
    RLCS_ERR_CAPTURE = 9     /* rlcs_gae_no_alloc: a device's first call was made while its stream was capturing */
} rlcs_status_t;

/* Human-readable name of a status code (static storage, never NULL). */
const char* rlcs_status_string(int status);

/* Bytes of workspace sufficient for any entry point at this (N, T); 0 when no row can straddle a
 * tile (then `workspace` may be NULL).  Returns 0 for invalid sizes as well. */
size_t rlcs_workspace_bytes(int64_t N, int64_t T);

/* Prepare a workspace (zero the tile records, set the call counter): enqueued on `cuda_stream`.
 * Needed once per workspace buffer, not once per call. */
int rlcs_workspace_init(void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Synchronises `cuda_stream`, reads the workspace's device status word and clears it.  Returns
 * RLCS_OK, RLCS_ERR_TIMEOUT, or RLCS_ERR_CUDA if the copy failed.  NULL workspace returns RLCS_OK. */
int rlcs_last_device_status(void* workspace, void* cuda_stream);

/*
 * Generalized Advantage Estimation -- Section 3.3.1, Table 1 row "GAE", boundaries of Section 3.2.
 *   delta_t = rewards_t + gamma * values_next(t) - values_t
 *   A_t     = delta_t + (cont_t ? gamma*lambda * A_{t+1} : 0)           (boundary carry A_T = 0)
 *   advantages[n,t] = A_t;   returns[n,t] = A_t + values_t   (returns may be NULL)
 * rewards, values, dones: [N,T]; truncs, trunc_bootstrap: [N,T] or NULL; bootstrap: [N] or NULL.
 */
int rlcs_gae(const float* rewards, const float* values, const uint8_t* dones, const uint8_t* truncs,
             const float* trunc_bootstrap, const float* bootstrap, float* advantages, float* returns,
             int64_t N, int64_t T, float gamma, float lambda,
             void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * GAE followed by advantage normalisation, the step directly downstream of GAE in PPO-style
 * training.  Section 9.3 lists "fused advantage normalization" as a planned extension without
 * defining it; the convention taken here is the usual one, over all N*T steps of the call:
 *   advantages[n,t] = (A_t - mean(A)) / (std(A) + eps),   std = sqrt(sum (A - mean)^2 / (N*T - ddof)),
 *   ddof = 0 (population) or 1 (sample; std = 0 when N*T = 1);   eps >= 0, finite
 *   returns[n,t]    = A_t + values_t  from the un-normalised A_t  (may be NULL)
 *   With eps = 0 and std = 0 (all advantages equal) the quotient is 0/0 and the advantages come out
 *   non-finite, as the formula says; pass eps > 0 to get zeros there.
 * Three launches: the GAE kernel (which also leaves, per tile, the sum of A and the sum of squared
 * deviations from the tile's own mean), a one-block reduction in double to mean and 1/(std + eps)
 * (the centred tile statistics are merged in double as sum(q_i + s_i^2 / n_i) - S^2 / (N*T), which
 * keeps a relative accuracy of about 2^-52 (mean / std)^2: a mean a thousand times the spread does
 * not cancel the variance away), and an in-place rescale of `advantages` -- one read of A
 * fewer than GAE, a statistics pass and a rescale.  Deterministic (fixed reduction order).
 * `workspace`: at least rlcs_gae_normalized_workspace_bytes(N, T) bytes (always > 0), 16-byte
 * aligned, initialised once with rlcs_workspace_init; same sharing rules as any workspace.
 */
int rlcs_gae_normalized(const float* rewards, const float* values, const uint8_t* dones, const uint8_t* truncs,
                        const float* trunc_bootstrap, const float* bootstrap, float* advantages, float* returns,
                        int64_t N, int64_t T, float gamma, float lambda, float eps, int ddof,
                        void* workspace, size_t workspace_bytes, void* cuda_stream);

size_t rlcs_gae_normalized_workspace_bytes(int64_t N, int64_t T);

/*
 * V-Trace -- Section 3.3.2, Table 1 row "V-Trace".  log_rhos[n,t] = log pi(a_t|s_t) - log mu(a_t|s_t).
 *   rho_t = min(rho_bar, exp(log_rhos_t));   c_t = min(c_bar, exp(log_rhos_t))
 *   Delta_t = rho_t*(rewards_t + gamma*values_next(t) - values_t) + (cont_t ? gamma*c_t*Delta_{t+1} : 0)
 *   vs[n,t] = values_t + Delta_t                                        (boundary carry Delta_T = 0)
 *   pg_advantages[n,t] = rho_t*(rewards_t + gamma*v_next - values_t),  v_next = cont_t ? vs_{t+1}
 *                        : values_next(t)                               (pg_advantages may be NULL)
 */
int rlcs_vtrace(const float* rewards, const float* values, const float* log_rhos, const uint8_t* dones,
                const uint8_t* truncs, const float* trunc_bootstrap, const float* bootstrap,
                float* vs, float* pg_advantages, int64_t N, int64_t T, float gamma, float rho_bar,
                float c_bar, void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Retrace(lambda) -- Section 3.3.3, Table 1 row "Retrace".  q_sa[n,t] = Q(s_t,a_t);
 * expected_q[n,t] = E_pi Q(s_t,.) (column 0 is never read); bootstrap[n] = E_pi Q(s_T,.).
 *   c_t = lambda * min(c_bar, exp(log_rhos_t))
 *   Delta_t = rewards_t + gamma*expected_q_next(t) - q_sa_t + (cont_t ? gamma*c_{t+1}*Delta_{t+1} : 0)
 *   q_targets[n,t] = q_sa_t + Delta_t          (index shift: the decay uses the NEXT step's c;
 *                                               Delta_T = 0 and log_rhos[n,T] is never needed)
 */
int rlcs_retrace(const float* rewards, const float* q_sa, const float* expected_q, const float* log_rhos,
                 const uint8_t* dones, const uint8_t* truncs, const float* trunc_bootstrap,
                 const float* bootstrap, float* q_targets, int64_t N, int64_t T, float gamma,
                 float lambda, float c_bar, void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Retrace(lambda) from the tensors a Q-learning agent holds -- Section 3.3.3 with the input form of
 * Section 7.3 (the paper's fused kernel reads the [N,T,A] action-probability tensor; its exact
 * signature is not given, this is the reading taken):
 *   q_values[n,t,a]        = Q(s_t, a)              target_probs[n,t,a]    = pi(a | s_t)
 *   behaviour_probs[n,t,a] = mu(a | s_t) (> 0 at the action taken)         actions[n,t] in [0, A), int32
 *   Q(s_t,a_t) = q_values[n,t,actions[n,t]];   E_pi Q(s_t,.) = sum_a target_probs[n,t,a] * q_values[n,t,a];
 *   c_t = lambda * min(c_bar, target_probs[n,t,a_t] / behaviour_probs[n,t,a_t])
 * and then exactly rlcs_retrace's recurrence and boundary rules (bootstrap[n] = E_pi Q(s_T,.),
 * trunc_bootstrap[n,t] = the continuation E_pi Q at a truncation).  [N,T,A] tensors are contiguous
 * with a innermost.  Only three scalars per step stay on chip, so the kernel's register need does
 * not depend on T.  Rows are read with 256-bit loads when A is 4, 8 or 16 and the three [N,T,A]
 * pointers are 32-byte aligned (for A = 4 and 8 the mu rows are read whole as well: a gather would
 * touch every sector anyway).  Actions outside [0, A) are clamped (for memory safety only).
 * The tile is 1024 steps: longer rows carry between thread blocks through the workspace's records,
 * except rows of whole tiles with A = 4 or 8 and about three rows per SM or more, which one thread
 * block each walks with the carry in a register (results agree to rounding).
 */
int rlcs_retrace_probs(const float* rewards, const float* q_values, const float* target_probs,
                       const float* behaviour_probs, const int32_t* actions, const uint8_t* dones, const uint8_t* truncs,
                       const float* trunc_bootstrap, const float* bootstrap, float* q_targets, int64_t N, int64_t T,
                       int64_t A, float gamma, float lambda, float c_bar,
                       void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * TD(lambda) returns -- Section 3.3.4, Table 1 row "TD(lambda)".
 *   G_t = rewards_t + gamma*[(1-lambda)*values_next(t) + lambda*G_{t+1}]     where cont_t,
 *   G_t = rewards_t + gamma*values_next(t)                                    elsewhere
 * (the window-edge bootstrap is priced once: gamma*(1-lambda) in alpha_{T-1} plus gamma*lambda
 * through the carry G_T = bootstrap).
 */
int rlcs_td_lambda(const float* rewards, const float* values, const uint8_t* dones, const uint8_t* truncs,
                   const float* trunc_bootstrap, const float* bootstrap, float* returns,
                   int64_t N, int64_t T, float gamma, float lambda,
                   void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Discounted returns -- Section 3.3.4 (lambda = 1, no value function), Table 1 row "Disc. Returns".
 *   G_t = rewards_t + gamma * (cont_t ? G_{t+1} : 0 | trunc_bootstrap_t | bootstrap per Section 3.2)
 */
int rlcs_discounted_return(const float* rewards, const uint8_t* dones, const uint8_t* truncs,
                           const float* trunc_bootstrap, const float* bootstrap, float* returns,
                           int64_t N, int64_t T, float gamma,
                           void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Eligibility trace, scalar per step, forward in time -- Section 3.3.5.
 *   z_t = x_t + ((t > 0 and not dones_{t-1}) ? gamma*lambda * z_{t-1} : 0)
 */
int rlcs_elig_trace(const float* x, const uint8_t* dones, float* traces, int64_t N, int64_t T,
                    float gamma, float lambda,
                    void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Vector-valued eligibility trace -- Table 1, row "Elig. Traces" in its vector form (Section 3.3.5):
 * x, traces: [N, T, D] contiguous with d innermost; one scalar decay per step, shared by all D
 * components;  dones: [N, T], the combined flag as for rlcs_elig_trace.
 *   z_t = x_t + ((t > 0 and not dones_{t-1}) ? gamma*lambda * z_{t-1} : 0)        (z_t, x_t in R^D)
 * One pass over x when N*D is large enough to fill the GPU; otherwise the time axis is cut into
 * chunks.  Where rows of D floats can be copied in 16-byte pieces (D a multiple of 4, D >= 32, x
 * 16-byte aligned) one launch chains the chunks: each is walked once from carry 0, and the steps
 * before its first cut are finished when the carry arrives from the records of the chunks before (a
 * bounded wait, as for the time-major entry points below), so x is still read once; otherwise three
 * launches read x twice (chunk ends, ordered carry chain, rescan).  Either way the result does not
 * depend on timing.  A cut needs `workspace` of
 * rlcs_elig_trace_vec_workspace_bytes(N, T, D) bytes (0 when no cut is needed; no initialisation
 * required for the results; the status word is as described for the time-major entry points).  128-bit accesses when D is a multiple of 4 and x, traces are 16-byte aligned.
 * Limits: T < 2^31, D <= 2^24, N*T*D < 2^40.
 */
int rlcs_elig_trace_vec(const float* x, const uint8_t* dones, float* traces, int64_t N, int64_t T, int64_t D,
                        float gamma, float lambda, void* workspace, size_t workspace_bytes, void* cuda_stream);

size_t rlcs_elig_trace_vec_workspace_bytes(int64_t N, int64_t T, int64_t D);

/*
 * Eligibility trace with a decay per component and step (the per-dimension beta_t that Section 9.1
 * lists as unsupported by a scalar-beta kernel; Eq. 1 component by component):
 *   z_t[c] = x_t[c] + ((t > 0 and not dones_{t-1}) ? beta_t[c] * z_{t-1}[c] : 0)
 * x, beta, traces: [N, T, D] contiguous with d innermost (beta[n, 0, :] is never used); dones [N, T].
 * Any finite beta is accepted (the caller folds gamma*lambda in).  Same kernel structure, workspace
 * rules (rlcs_elig_trace_vec_beta_workspace_bytes), alignment rules and limits as rlcs_elig_trace_vec.
 */
int rlcs_elig_trace_vec_beta(const float* x, const float* beta, const uint8_t* dones, float* traces, int64_t N, int64_t T,
                             int64_t D, void* workspace, size_t workspace_bytes, void* cuda_stream);

size_t rlcs_elig_trace_vec_beta_workspace_bytes(int64_t N, int64_t T, int64_t D);

/*
 * Episodic prefix sum, forward in time -- Section 3.3.6.
 *   starts_at == 0 ("ends_at", the flag closes a segment):  C_t = x_t + ((t>0 and not dones_{t-1}) ? C_{t-1} : 0)
 *   starts_at != 0 (the flag opens a segment):              C_t = x_t + ((t>0 and not dones_t)     ? C_{t-1} : 0)
 */
int rlcs_episodic_prefix_sum(const float* x, const uint8_t* dones, float* sums, int64_t N, int64_t T,
                             int starts_at, void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * GAE without any workspace argument, for callers that cannot allocate device memory.  (The paper
 * has no counterpart: its library allocates through PyTorch.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a stream capture or other
 * region in which the driver refuses allocation, in a process whose memory was handed out
 * completely to a pool up front, or in a real-time control loop that must not take the allocator's
 * locks -- and that cannot carve a workspace for rlcs_gae out of memory it already owns.  Same
 * arguments and results as rlcs_gae; the scratch for the carry between thread blocks lives in a
 * fixed 1 MiB device array inside the library (rlcs_no_alloc_scratch_bytes()), which every GPU
 * that loads the library holds until the process exits.  The call itself allocates nothing: no
 * cudaMalloc, no cudaFree, no allocating library routine.
 *
 * Limit: the carry scratch this call would use, rlcs_gae_carry_bytes(N, T, truncs != NULL, all
 * pointers aligned for vector access), must not exceed that array.  That always holds for
 * N*T <= 33 545 728 steps (65 520 tile records of at least 512 steps), and for any size when no
 * row straddles a tile (T divides the tile, e.g. 16384 x 2048) or the tiles of a row form one
 * thread-block cluster.  Larger problems return RLCS_ERR_LIMIT and launch nothing.
 * First call on a device: looks up the array's device address (cudaGetSymbolAddress) and
 * initialises it with two small memsets on `cuda_stream`; make this first call outside any stream
 * capture (it returns RLCS_ERR_CAPTURE otherwise, since the memsets would be recorded instead of
 * run), with the device current that later calls will use.  Concurrent first calls from several
 * host threads are serialised by a lock; later calls take it only to read the cached address.
 * Sharing: every call on a device uses the same array, which keeps what the last call left; the
 * entry point re-zeroes the word that must start at zero.  Calls that can overlap on the GPU
 * (different streams without ordering, several host threads) race on it and give wrong results:
 * keep them ordered, or use rlcs_gae with separate workspaces.
 * Device status: a bounded carry wait that gave up leaves RLCS_ERR_TIMEOUT in the array's status
 * word, where it stays until rlcs_no_alloc_last_device_status reads and clears it.
 */
int rlcs_gae_no_alloc(const float* rewards, const float* values, const uint8_t* dones, const uint8_t* truncs,
                      const float* trunc_bootstrap, const float* bootstrap, float* advantages, float* returns,
                      int64_t N, int64_t T, float gamma, float lambda, void* cuda_stream);

/* Device status of the rlcs_gae_no_alloc calls on the current device, like rlcs_last_device_status
 * for a workspace: synchronises `cuda_stream`, returns RLCS_OK or RLCS_ERR_TIMEOUT and clears the
 * word.  RLCS_OK when rlcs_gae_no_alloc has not run on this device yet.  (No counterpart in the paper.) */
int rlcs_no_alloc_last_device_status(void* cuda_stream);

/* Bytes of carry workspace one rlcs_gae call with these sizes would read or write: 0 when no row
 * straddles a tile or a row's tiles form one thread-block cluster (needs `vector_access`: every fp32
 * pointer 32-byte and every mask pointer 16-byte aligned); never more than rlcs_workspace_bytes(N, T),
 * which stays the size to allocate for a workspace shared by all entry points. */
size_t rlcs_gae_carry_bytes(int64_t N, int64_t T, int has_truncs, int vector_access);

/* Size in bytes of the built-in scratch array used by rlcs_gae_no_alloc. */
size_t rlcs_no_alloc_scratch_bytes(void);

/*
 * Time-major variants of the seven entry points: every [T, N] tensor has element (t, n) at t*N + n
 * (step-major rollout storage); `bootstrap` stays [N].  Same definitions, flags, NULL conventions and
 * parameter checks as the row-major entry points above; only the layout differs.  (The paper's API
 * is row-major only; time-major buffers are what step-major collectors hold, cf. Section 9.1.)
 * A lane per environment walks its timesteps in scan order.  When N is a multiple of 16 and the
 * per-step inputs are 16-byte aligned each warp streams its 32 columns through a shared-memory ring
 * of asynchronous copies; otherwise the same walk runs from registers (any N, 4-byte alignment).
 * When N alone cannot fill the GPU the time axis is cut into chunks.  On the ring path one launch
 * chains them: thread blocks take (column block, chunk) pairs in scan order from a ticket counter,
 * walk their chunk for its aggregate, obtain the carry into it from the records of the chunks before
 * (a bounded wait) and walk it again from L2 to write the outputs; on the register path three
 * launches read the inputs twice (chunk aggregates, ordered carry chain, second walk).  Either way
 * the result does not depend on timing.  Both need `workspace` of
 * rlcs_time_major_workspace_bytes(N, T) bytes (0 when no cut is needed): 16-byte aligned; its
 * contents need no initialisation for the results, but word 2 is a status word like that of the
 * row-major workspaces (set to RLCS_ERR_TIMEOUT when a wait ran out, read and cleared by
 * rlcs_last_device_status), so zero the first 256 bytes once -- rlcs_workspace_init does -- if you
 * intend to query it.  Calls that may overlap on the GPU need separate workspaces.
 */
size_t rlcs_time_major_workspace_bytes(int64_t N, int64_t T);
int rlcs_gae_time_major(const float* rewards, const float* values, const uint8_t* dones, const uint8_t* truncs,
                        const float* trunc_bootstrap, const float* bootstrap, float* advantages, float* returns,
                        int64_t N, int64_t T, float gamma, float lambda,
                        void* workspace, size_t workspace_bytes, void* cuda_stream);
int rlcs_vtrace_time_major(const float* rewards, const float* values, const float* log_rhos, const uint8_t* dones,
                           const uint8_t* truncs, const float* trunc_bootstrap, const float* bootstrap, float* vs,
                           float* pg_advantages, int64_t N, int64_t T, float gamma, float rho_bar, float c_bar,
                           void* workspace, size_t workspace_bytes, void* cuda_stream);
int rlcs_retrace_time_major(const float* rewards, const float* q_sa, const float* expected_q, const float* log_rhos,
                            const uint8_t* dones, const uint8_t* truncs, const float* trunc_bootstrap,
                            const float* bootstrap, float* q_targets, int64_t N, int64_t T, float gamma, float lambda,
                            float c_bar, void* workspace, size_t workspace_bytes, void* cuda_stream);
int rlcs_td_lambda_time_major(const float* rewards, const float* values, const uint8_t* dones, const uint8_t* truncs,
                              const float* trunc_bootstrap, const float* bootstrap, float* returns, int64_t N,
                              int64_t T, float gamma, float lambda,
                              void* workspace, size_t workspace_bytes, void* cuda_stream);
int rlcs_discounted_return_time_major(const float* rewards, const uint8_t* dones, const uint8_t* truncs,
                                      const float* trunc_bootstrap, const float* bootstrap, float* returns, int64_t N,
                                      int64_t T, float gamma, void* workspace, size_t workspace_bytes, void* cuda_stream);
int rlcs_elig_trace_time_major(const float* x, const uint8_t* dones, float* traces, int64_t N, int64_t T, float gamma,
                               float lambda, void* workspace, size_t workspace_bytes, void* cuda_stream);
int rlcs_episodic_prefix_sum_time_major(const float* x, const uint8_t* dones, float* sums, int64_t N, int64_t T,
                                        int starts_at, void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * GAE with observation-skip masking (planned in Section 9.2: "carries the recurrence across masked
 * tokens (beta_t = 1)"; for token-level trajectories whose observation / tool tokens are not actions).
 * skip [N, T] uint8, non-zero = masked.  Reading: a masked step is transparent --
 *   masked t:    A_t = A_{t+1},  W_t = W_{t+1}                      (no TD error, no discount)
 *   unmasked t:  A_t = r_t + gamma*W_{t+1} - V_t + gamma*lambda*A_{t+1},  W_t = V_t
 * with A = 0 and W = bootstrap beyond the window, and termination / truncation flags severing both
 * recurrences as in rlcs_gae wherever they stand (at a flagged masked step A_t = 0 and W_t is the
 * flag's successor value).  Without flags on masked steps, the advantages at the unmasked steps are
 * rlcs_gae of the rows with the masked steps deleted.
 * Outputs: values_filled = W (required), advantages = A, returns = A + W (optional).  One launch:
 * per tile, W by a backward scan and then the masked GAE scan on (rewards, W), each with its own
 * carry between tiles (through the workspace's records; rows of whole 1024-step tiles with about
 * three rows per SM or more are walked by one thread block each, both carries in registers).
 * Same flags, NULL conventions, alignment rules and workspace as rlcs_gae.
 */
int rlcs_gae_skip(const float* rewards, const float* values, const uint8_t* dones, const uint8_t* truncs,
                  const float* trunc_bootstrap, const float* bootstrap, const uint8_t* skip, float* values_filled,
                  float* advantages, float* returns, int64_t N, int64_t T, float gamma, float lambda,
                  void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * bfloat16-tensor variants of the seven entry points (the paper's kernels are fp32-only; Section 9.1
 * defers bfloat16, Section 9.2 plans it): every float tensor -- inputs, trunc_bootstrap, bootstrap
 * and outputs -- holds bfloat16 bit patterns (uint16_t, row-major [N, T], 2-byte aligned; 32-byte
 * alignment of all of them enables vector access), masks stay uint8.  Inputs are widened to fp32 on
 * load (exact), all arithmetic and the carries between tiles are fp32, outputs are rounded to
 * nearest-even once, on store.  Same definitions, flags, NULL conventions, parameter checks and
 * workspace (rlcs_workspace_bytes, rlcs_workspace_init) as the fp32 entry points.
 */
int rlcs_gae_bf16(const uint16_t* rewards, const uint16_t* values, const uint8_t* dones, const uint8_t* truncs,
                  const uint16_t* trunc_bootstrap, const uint16_t* bootstrap, uint16_t* advantages, uint16_t* returns,
                  int64_t N, int64_t T, float gamma, float lambda,
                  void* workspace, size_t workspace_bytes, void* cuda_stream);
int rlcs_vtrace_bf16(const uint16_t* rewards, const uint16_t* values, const uint16_t* log_rhos, const uint8_t* dones,
                     const uint8_t* truncs, const uint16_t* trunc_bootstrap, const uint16_t* bootstrap, uint16_t* vs,
                     uint16_t* pg_advantages, int64_t N, int64_t T, float gamma, float rho_bar, float c_bar,
                     void* workspace, size_t workspace_bytes, void* cuda_stream);
int rlcs_retrace_bf16(const uint16_t* rewards, const uint16_t* q_sa, const uint16_t* expected_q, const uint16_t* log_rhos,
                      const uint8_t* dones, const uint8_t* truncs, const uint16_t* trunc_bootstrap,
                      const uint16_t* bootstrap, uint16_t* q_targets, int64_t N, int64_t T, float gamma, float lambda,
                      float c_bar, void* workspace, size_t workspace_bytes, void* cuda_stream);
int rlcs_td_lambda_bf16(const uint16_t* rewards, const uint16_t* values, const uint8_t* dones, const uint8_t* truncs,
                        const uint16_t* trunc_bootstrap, const uint16_t* bootstrap, uint16_t* returns, int64_t N,
                        int64_t T, float gamma, float lambda,
                        void* workspace, size_t workspace_bytes, void* cuda_stream);
int rlcs_discounted_return_bf16(const uint16_t* rewards, const uint8_t* dones, const uint8_t* truncs,
                                const uint16_t* trunc_bootstrap, const uint16_t* bootstrap, uint16_t* returns, int64_t N,
                                int64_t T, float gamma, void* workspace, size_t workspace_bytes, void* cuda_stream);
int rlcs_elig_trace_bf16(const uint16_t* x, const uint8_t* dones, uint16_t* traces, int64_t N, int64_t T, float gamma,
                         float lambda, void* workspace, size_t workspace_bytes, void* cuda_stream);
int rlcs_episodic_prefix_sum_bf16(const uint16_t* x, const uint8_t* dones, uint16_t* sums, int64_t N, int64_t T,
                                  int starts_at, void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Test hook: the bare scan of Eq. 1 / Eq. 2 on caller-supplied coefficients, every row with
 * boundary carry 0 (the paper's generic kernel of Section 4.1).
 *   forward == 0:  out_t = alpha_t + (t < T-1 ? beta_t * out_{t+1} : 0)
 *   forward != 0:  out_t = alpha_t + (t > 0   ? beta_t * out_{t-1} : 0)
 */
int rlcs_affine_scan(const float* alpha, const float* beta, float* out, int64_t N, int64_t T, int forward,
                     void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Test hook: choose the kernel and tile shape for subsequent calls in this process (not
 * thread-safe).  variant -1 = chosen per call from algorithm and problem size (the default).  Other variants change the kernel (persistent
 * blocks with a bulk-copy ring, or one tile per block), threads per block and steps per thread,
 * hence where tiles and warps cut the rows; results must agree across variants to rounding, and
 * exactly at severed steps.  Returns RLCS_ERR_ARG for an unknown variant.  rlcs_workspace_bytes is
 * an upper bound over all variants.
 */
int rlcs_debug_set_tile_variant(int variant);
/* 1 if that tile variant is compiled into this build (the default build holds the shapes the
 * selection can return plus two bulk-copy ring shapes; -DRLCS_ALL_VARIANTS compiles the whole table),
 * else 0.  rlcs_debug_set_tile_variant returns RLCS_ERR_ARG for a variant that is not compiled. */
int rlcs_debug_variant_built(int variant);

/* Elements per tile of a variant (0 for an unknown variant). */
int rlcs_debug_tile_elems(int variant);

/*
 * Which variant a call would use: algorithm 0 = GAE, 1 = TD(lambda), 2 = discounted return,
 * 3 = V-Trace, 4 = Retrace, 5 = eligibility trace, 6 = prefix sum, 7 / 8 = rlcs_affine_scan backward /
 * forward.  Honours rlcs_debug_set_tile_variant.  -1 for invalid arguments or an empty problem.
 */
int rlcs_debug_variant_for(int algorithm, int has_truncs, int64_t N, int64_t T);

/* Shape of a variant: threads per block, steps per thread, blocks per SM it is compiled for, and
 * ring stages (0 = the one-tile-per-block kernel).  Any output pointer may be NULL. */
int rlcs_debug_variant_info(int variant, int* threads, int* steps_per_thread, int* blocks_per_sm, int* ring_stages);

/* Test / measurement hook for the one-thread-block-per-row kernel (rows longer than a tile, T a
 * multiple of the steps per thread): -1 = used when there are at least as many rows as thread
 * blocks fit on the GPU (default), 0 = never, 1 = whenever legal.  Results agree to rounding. */
int rlcs_debug_set_row_blocks(int mode);

/* Test / measurement hook: 0 turns row-aligned tiling off (see "Workspace" above: rows shorter than a
 * tile that do not divide it are then carried between thread blocks through the workspace, as rows
 * longer than a tile always are), 1 (default) allows it.  Results agree to rounding. */
int rlcs_debug_allow_row_tiles(int on);

/* Test / measurement hook: 0 launches the row-major scan kernels without programmatic stream
 * serialisation (see "Execution" above), 1 (default) with it.  Results are identical. */
int rlcs_debug_set_dependent_launch(int on);

/*
 * Test hook: rows that are exactly 2..8 tiles long are scanned by one thread-block cluster per row,
 * with the carry between blocks in distributed shared memory (no workspace use).  on == 0 sends
 * such calls through the workspace look-back instead.  Results must agree to rounding.
 */
int rlcs_debug_allow_cluster_carry(int on);

/*
 * Test hook: with on != 0, subsequent calls compute row and timestep of a step with the 64-bit
 * arithmetic that problems of 2^32 steps and more need, whatever their size (the 32-bit path uses a
 * multiply-shift division by T).  Results must be identical.
 */
int rlcs_debug_force_wide_index(int on);

/*
 * Test hook for the bounded carry wait: for subsequent calls in this process, the thread block
 * whose scan-order index is `mute_tile` does not publish its tile record (negative = publish
 * normally), and the wait gives up after `spin_cap` polls (<= 0 = default).  A dependent block
 * then runs out of polls within microseconds, records RLCS_ERR_TIMEOUT in the workspace status
 * word and finishes normally -- nothing hangs or faults.  The chained time-major kernel (and the
 * vector traces that use it) honours both: there `mute_tile` is the ticket of the block that
 * publishes neither its chunk aggregate nor the value it carries out.
 */
int rlcs_debug_set_carry_fault(int64_t mute_tile, int64_t spin_cap);

/*
 * Test hook: path of the time-major entry points for subsequent calls in this process.  1 = the
 * register walk whatever the alignment; 3 = the shared-memory ring with one column per lane whatever
 * the size; 4 = a cut time axis always by three launches, never the chained kernel; 5 = the chained
 * kernel whenever T exceeds one of its chunks, also where N alone would fill the GPU (the workspace
 * query follows); any other value = the default (the ring wherever N and the pointers allow it, two
 * columns per lane for large N, the chained kernel where the time axis is cut).  Results must agree
 * to rounding.
 */
void rlcs_debug_time_major_path(int path);

/*
 * Test hook: plan of the vector-trace entry points for subsequent calls in this process.  batch = 8,
 * 16 or 32: the walk with one thread per component group and that many timesteps loaded ahead;
 * batch = 1: the time-major block kernel wherever its copies can be issued; any other value: planned
 * from N, T and D.  chunks > 0 (with the walk)
 * cuts every row's time axis into that many chunks (capped by the minimum chunk length; 1 = never
 * cut; <= 0: planned).  The *_workspace_bytes queries follow the forced plan.  Results must agree to
 * rounding.
 */
void rlcs_debug_vec_trace_plan(int batch, int chunks);

/*
 * Measurement hook: a streaming kernel that reads read_bytes from src and writes write_bytes to dst
 * (whole 32-byte pieces; both pointers 32-byte aligned, buffers at least that large; dst[0] may be
 * written when write_bytes is 0), with the scan kernels' load / store instructions and one piece
 * per thread.  bench.py times it at a scan launch's byte count and read:write ratio to report the
 * bandwidth ceiling of that size next to the scan's own figure.
 */
int rlcs_debug_stream_copy(const float* src, float* dst, size_t read_bytes, size_t write_bytes, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* RLCS_H_ */
