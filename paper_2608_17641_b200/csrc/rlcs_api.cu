// C ABI of the library: argument validation, kernel selection, launch.  No allocation, no state
// between calls apart from the two test hooks at the bottom.
#include "rlcs_host.cuh"

namespace rlcs_hooks {
int g_variant = -1;
bool g_cluster = true;
bool g_wide_index = false;
long long g_mute_tile = -1;
long long g_spin_cap = 0;
bool g_pdl = true;
bool g_row_tiles = true;
int g_row_blocks = -1;
}  // namespace rlcs_hooks

extern "C" {

const char* rlcs_status_string(int status) {
    switch (status) {
        case RLCS_OK: return "RLCS_OK";
        case RLCS_ERR_NULL: return "RLCS_ERR_NULL: required pointer is NULL (or only one of truncs/trunc_bootstrap given)";
        case RLCS_ERR_SIZE: return "RLCS_ERR_SIZE: N or T negative or too large";
        case RLCS_ERR_ARG: return "RLCS_ERR_ARG: gamma/lambda/clip out of range";
        case RLCS_ERR_ALIGN: return "RLCS_ERR_ALIGN: misaligned pointer";
        case RLCS_ERR_WORKSPACE: return "RLCS_ERR_WORKSPACE: workspace missing or too small";
        case RLCS_ERR_CUDA: return "RLCS_ERR_CUDA: CUDA call failed";
        case RLCS_ERR_TIMEOUT: return "RLCS_ERR_TIMEOUT: bounded carry wait gave up";
        case RLCS_ERR_LIMIT: return "RLCS_ERR_LIMIT: problem too large for the built-in scratch array of rlcs_gae_no_alloc";
        case RLCS_ERR_CAPTURE: return "RLCS_ERR_CAPTURE: first rlcs_gae_no_alloc call on a device made during stream capture";
        default: return "RLCS: unknown status";
    }
}

size_t rlcs_workspace_bytes(int64_t N, int64_t T) {
    int64_t total = 0;
    if (check_sizes(N, T, &total) != RLCS_OK || total == 0) return 0;
    if (rlcs::kMinTileElems % T == 0) return 0;     // T divides every tile size: no row straddles a tile
    // one record per 512-step tile, plus one: rlcs_gae_skip keeps two records per tile of >= 1024 steps
    const int64_t tiles = (total + rlcs::kMinTileElems - 1) / rlcs::kMinTileElems;
    return sizeof(unsigned) * rlcs::kHeaderWords + sizeof(uint4) * (size_t)(tiles + 1);
}

int rlcs_workspace_init(void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (workspace == nullptr) return workspace_bytes == 0 ? RLCS_OK : RLCS_ERR_NULL;
    if (!aligned(workspace, 16)) return RLCS_ERR_ALIGN;
    if (workspace_bytes < sizeof(unsigned) * rlcs::kHeaderWords) return RLCS_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    if (cudaMemsetAsync(workspace, 0, workspace_bytes, s) != cudaSuccess) return RLCS_ERR_CUDA;
    // the call counter starts at 256 (byte pattern 0x00 0x01 0x00 0x00): zeroed records are never
    // valid, and neither are the small record tags (0, 1, 2) that the time-major kernels leave in the
    // same area when a workspace is shared between the two families of entry points
    if (cudaMemsetAsync(static_cast<unsigned char*>(workspace) + 1, 1, 1, s) != cudaSuccess) return RLCS_ERR_CUDA;
    return RLCS_OK;
}

int rlcs_last_device_status(void* workspace, void* cuda_stream) {
    if (workspace == nullptr) return RLCS_OK;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    unsigned status = 0;
    unsigned* word = static_cast<unsigned*>(workspace) + 2;
    if (cudaMemcpyAsync(&status, word, sizeof(status), cudaMemcpyDeviceToHost, s) != cudaSuccess) return RLCS_ERR_CUDA;
    if (cudaMemsetAsync(word, 0, sizeof(status), s) != cudaSuccess) return RLCS_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return RLCS_ERR_CUDA;
    return status == 0 ? RLCS_OK : (int)status;
}

int rlcs_gae(const float* rewards, const float* values, const uint8_t* dones, const uint8_t* truncs,
             const float* trunc_bootstrap, const float* bootstrap, float* advantages, float* returns,
             int64_t N, int64_t T, float gamma, float lambda, void* workspace, size_t workspace_bytes,
             void* cuda_stream) {
    ScanParams p = {};
    Ptrs ps;
    int64_t total;
    bool vec;
    if (!unit_interval(gamma) || !unit_interval(lambda)) return RLCS_ERR_ARG;
    ps.add_f32(rewards); ps.add_f32(values); ps.add_f32(advantages); ps.add_f32(returns);
    int st = backward_common(p, ps, dones, truncs, trunc_bootstrap, bootstrap, N, T, &total, &vec);
    if (st != RLCS_OK || total == 0) return st;
    if (!rewards || !values || !advantages) return RLCS_ERR_NULL;
    p.f0 = rewards; p.f1 = values; p.out0 = advantages; p.out1 = returns;
    p.gamma = gamma; p.decay = gamma * lambda;
    const int variant = choose_variant(rlcs::kGae, truncs != nullptr, total, T);
    st = finish_params(p, variant, total, T, workspace, workspace_bytes, vec);
    if (st != RLCS_OK) return st;
    return run(rlcs::launch_gae, p, variant, truncs != nullptr, vec, cuda_stream);
}

size_t rlcs_gae_carry_bytes(int64_t N, int64_t T, int has_truncs, int vector_access) {
    int64_t total = 0;
    if (check_sizes(N, T, &total) != RLCS_OK || total == 0) return 0;
    const int variant = choose_variant(rlcs::kGae, has_truncs != 0, total, T);
    return plan_carry(variant, total, T, vector_access != 0, true, 1).bytes;
}

int rlcs_gae_skip(const float* rewards, const float* values, const uint8_t* dones, const uint8_t* truncs,
                  const float* trunc_bootstrap, const float* bootstrap, const uint8_t* skip, float* values_filled,
                  float* advantages, float* returns, int64_t N, int64_t T, float gamma, float lambda, void* workspace,
                  size_t workspace_bytes, void* cuda_stream) {
    ScanParams p = {};
    Ptrs ps;
    int64_t total;
    bool vec;
    if (!unit_interval(gamma) || !unit_interval(lambda)) return RLCS_ERR_ARG;
    ps.add_f32(rewards); ps.add_f32(values); ps.add_f32(values_filled); ps.add_f32(advantages); ps.add_f32(returns);
    ps.add_u8(skip);
    int st = backward_common(p, ps, dones, truncs, trunc_bootstrap, bootstrap, N, T, &total, &vec);
    if (st != RLCS_OK || total == 0) return st;
    if (!rewards || !values || !skip || !values_filled || !advantages) return RLCS_ERR_NULL;
    p.skip = skip;
    p.gamma = gamma; p.decay = gamma * lambda;
    p.f0 = rewards; p.f1 = values; p.out2 = values_filled; p.out0 = advantages; p.out1 = returns;
    // One launch runs both scans per tile (value fill, then the masked GAE on its result); each scan has
    // its own carry records.  These tile shapes have at least 1024 steps, so two records per tile still
    // fit the workspace of rlcs_workspace_bytes (sized for 512-step tiles).  No cluster carry here.
    int variant = choose_variant(rlcs::kGaeSkip, truncs != nullptr, total, T);
    // Rows of whole tiles, about three per SM or more: one thread block per row, both carries in
    // registers (token-level trajectories are long).  Measured at 4096 x 8192 / 1024 x 32768, fraction of
    // the copy bandwidth: records through the workspace 0.68 / 0.62; rows with 128 x 16 tiles at 5 / 6 / 8
    // blocks per SM 0.84 / 0.70, 0.80 / 0.63, 0.58 / 0.55; 256 x 8 0.89 / 0.81; 128 x 8 at 8 blocks 0.90 / 0.85.
    constexpr int kRowsVariant = 6;
    if (rlcs_hooks::g_variant < 0 && T > 2048 && T % tile_elems(kRowsVariant) == 0 && row_blocks_ok(kRowsVariant, total, T, vec, true))
        variant = kRowsVariant;
    const bool rows_ok = T % tile_elems(variant) == 0;
    st = finish_params(p, variant, total, T, workspace, workspace_bytes, vec, false, 2, false, rows_ok ? 2 : 0);
    if (st != RLCS_OK) return st;
    return run(rlcs::launch_gae_skip, p, variant, truncs != nullptr, vec, cuda_stream);
}

// Layout of the workspace of rlcs_gae_normalized: the carry workspace of rlcs_workspace_bytes (rounded
// up to 256 bytes), then {mean, 1/(std+eps)} in a 256-byte slot, then one {sum, sum of squares} pair per tile.
static size_t norm_carry_bytes(int64_t N, int64_t T) { return (rlcs_workspace_bytes(N, T) + 255) / 256 * 256; }

size_t rlcs_gae_normalized_workspace_bytes(int64_t N, int64_t T) {
    int64_t total = 0;
    if (check_sizes(N, T, &total) != RLCS_OK || total == 0) return 0;
    const int64_t tiles = (total + rlcs::kMinTileElems - 1) / rlcs::kMinTileElems;
    return norm_carry_bytes(N, T) + 256 + 2 * sizeof(float) * (size_t)tiles;
}

int rlcs_gae_normalized(const float* rewards, const float* values, const uint8_t* dones, const uint8_t* truncs,
                        const float* trunc_bootstrap, const float* bootstrap, float* advantages, float* returns,
                        int64_t N, int64_t T, float gamma, float lambda, float eps, int ddof, void* workspace,
                        size_t workspace_bytes, void* cuda_stream) {
    ScanParams p = {};
    Ptrs ps;
    int64_t total;
    bool vec;
    if (!unit_interval(gamma) || !unit_interval(lambda) || !(eps >= 0.f) || std::isinf(eps) || (ddof != 0 && ddof != 1))
        return RLCS_ERR_ARG;
    ps.add_f32(rewards); ps.add_f32(values); ps.add_f32(advantages); ps.add_f32(returns);
    int st = backward_common(p, ps, dones, truncs, trunc_bootstrap, bootstrap, N, T, &total, &vec);
    if (st != RLCS_OK || total == 0) return st;
    if (!rewards || !values || !advantages) return RLCS_ERR_NULL;
    if (workspace == nullptr || workspace_bytes < rlcs_gae_normalized_workspace_bytes(N, T)) return RLCS_ERR_WORKSPACE;
    if (!aligned(workspace, 16)) return RLCS_ERR_ALIGN;
    const size_t carry_bytes = norm_carry_bytes(N, T);
    float* mean_rstd = reinterpret_cast<float*>(static_cast<unsigned char*>(workspace) + carry_bytes);
    p.f0 = rewards; p.f1 = values; p.out0 = advantages; p.out1 = returns;
    p.stats = mean_rstd + 64;
    p.gamma = gamma; p.decay = gamma * lambda;
    const int variant = choose_variant(rlcs::kGaeStats, truncs != nullptr, total, T);
    // (the statistics flavour keeps fixed tiles: its per-tile sums are laid out for them; rows of whole
    // tiles, about three per SM or more, take one thread block per row like plain GAE)
    // (1024 x 32768, a thin second wave of blocks: 0.75 with one block per row against 0.80 with the carry
    // between blocks -- plan_carry's rule keeps such shapes off the row kernel)
    const bool rows_ok = T % tile_elems(variant) == 0;
    st = finish_params(p, variant, total, T, carry_bytes ? workspace : nullptr, carry_bytes, vec, true, 1, false, rows_ok ? 1 : 0);
    if (st != RLCS_OK) return st;
    st = run(rlcs::launch_gae_stats, p, variant, truncs != nullptr, vec, cuda_stream);
    if (st != RLCS_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const long long stat_tiles = p.row_blocks ? (total / T) * (T / tile_elems(variant)) : p.num_tiles;   // one pair of sums per tile
    if (rlcs::launch_norm_finalize(p.stats, stat_tiles, total, (int)p.tile_steps, ddof, eps, mean_rstd, s) != cudaSuccess) return RLCS_ERR_CUDA;
    if (rlcs::launch_norm_rescale(advantages, total, mean_rstd, vec, s) != cudaSuccess) return RLCS_ERR_CUDA;
    return RLCS_OK;
}

int rlcs_vtrace(const float* rewards, const float* values, const float* log_rhos, const uint8_t* dones,
                const uint8_t* truncs, const float* trunc_bootstrap, const float* bootstrap, float* vs,
                float* pg_advantages, int64_t N, int64_t T, float gamma, float rho_bar, float c_bar,
                void* workspace, size_t workspace_bytes, void* cuda_stream) {
    ScanParams p = {};
    Ptrs ps;
    int64_t total;
    bool vec;
    if (!unit_interval(gamma) || !clip_ok(rho_bar) || !clip_ok(c_bar)) return RLCS_ERR_ARG;
    ps.add_f32(rewards); ps.add_f32(values); ps.add_f32(log_rhos); ps.add_f32(vs); ps.add_f32(pg_advantages);
    int st = backward_common(p, ps, dones, truncs, trunc_bootstrap, bootstrap, N, T, &total, &vec);
    if (st != RLCS_OK || total == 0) return st;
    if (!rewards || !values || !log_rhos || !vs) return RLCS_ERR_NULL;
    p.f0 = rewards; p.f1 = values; p.f3 = log_rhos; p.out0 = vs; p.out1 = pg_advantages;
    p.gamma = gamma; p.rho_bar = rho_bar; p.c_bar = c_bar;
    const int variant = choose_variant(rlcs::kVtrace, truncs != nullptr, total, T);
    st = finish_params(p, variant, total, T, workspace, workspace_bytes, vec);
    if (st != RLCS_OK) return st;
    return run(rlcs::launch_vtrace, p, variant, truncs != nullptr, vec, cuda_stream);
}

int rlcs_retrace(const float* rewards, const float* q_sa, const float* expected_q, const float* log_rhos,
                 const uint8_t* dones, const uint8_t* truncs, const float* trunc_bootstrap,
                 const float* bootstrap, float* q_targets, int64_t N, int64_t T, float gamma, float lambda,
                 float c_bar, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    ScanParams p = {};
    Ptrs ps;
    int64_t total;
    bool vec;
    if (!unit_interval(gamma) || !unit_interval(lambda) || !clip_ok(c_bar)) return RLCS_ERR_ARG;
    ps.add_f32(rewards); ps.add_f32(q_sa); ps.add_f32(expected_q); ps.add_f32(log_rhos); ps.add_f32(q_targets);
    int st = backward_common(p, ps, dones, truncs, trunc_bootstrap, bootstrap, N, T, &total, &vec);
    if (st != RLCS_OK || total == 0) return st;
    if (!rewards || !q_sa || !expected_q || !log_rhos || !q_targets) return RLCS_ERR_NULL;
    p.f0 = rewards; p.f1 = q_sa; p.f2 = expected_q; p.f3 = log_rhos; p.out0 = q_targets;
    p.gamma = gamma; p.aux = gamma * lambda; p.c_bar = c_bar;
    const int variant = choose_variant(rlcs::kRetrace, truncs != nullptr, total, T);
    st = finish_params(p, variant, total, T, workspace, workspace_bytes, vec);
    if (st != RLCS_OK) return st;
    return run(rlcs::launch_retrace, p, variant, truncs != nullptr, vec, cuda_stream);
}

int rlcs_retrace_probs(const float* rewards, const float* q_values, const float* target_probs,
                       const float* behaviour_probs, const int32_t* actions, const uint8_t* dones, const uint8_t* truncs,
                       const float* trunc_bootstrap, const float* bootstrap, float* q_targets, int64_t N, int64_t T,
                       int64_t A, float gamma, float lambda, float c_bar, void* workspace, size_t workspace_bytes,
                       void* cuda_stream) {
    ScanParams p = {};
    Ptrs ps;
    int64_t total;
    bool vec;
    if (!unit_interval(gamma) || !unit_interval(lambda) || !clip_ok(c_bar)) return RLCS_ERR_ARG;
    if (A < 1 || A > (int64_t(1) << 20)) return RLCS_ERR_SIZE;
    ps.add_f32(rewards); ps.add_f32(q_targets);
    int st = backward_common(p, ps, dones, truncs, trunc_bootstrap, bootstrap, N, T, &total, &vec);
    if (st != RLCS_OK || total == 0) return st;
    if (total > kMaxTotal / A) return RLCS_ERR_SIZE;
    if (!rewards || !q_values || !target_probs || !behaviour_probs || !actions || !q_targets) return RLCS_ERR_NULL;
    if (!aligned(q_values, 4) || !aligned(target_probs, 4) || !aligned(behaviour_probs, 4) || !aligned(actions, 4))
        return RLCS_ERR_ALIGN;
    const bool vec_rows = (A % 4 == 0) && aligned(q_values, 32) && aligned(target_probs, 32) && aligned(behaviour_probs, 32);
    p.f0 = rewards; p.f1 = q_values; p.pi = target_probs; p.mu = behaviour_probs; p.actions = actions; p.A = (int)A;
    p.out0 = q_targets;
    p.gamma = gamma; p.aux = gamma * lambda; p.c_bar = c_bar;
    constexpr int kVariant = 3;      // 256 threads x 4 steps, the tile rlcs_retrace_probs.cu instantiates
    static_assert(rlcs::kVariants[kVariant].threads == rlcs::kRetraceProbsThreads &&
                  rlcs::kVariants[kVariant].items == rlcs::kRetraceProbsItems, "tile shape mismatch");
    // One thread block per row where rows are whole tiles and there are enough of them (no carry between
    // blocks): measured at 16384 x 2048 / 8192 x 4096 / 2048 x 16384 against the carry through tile records,
    // fraction of the copy bandwidth: A = 4 0.86 -> 0.92 / 0.95 / 0.91, A = 8 0.87 / 0.84 / 0.81 -> 0.94 /
    // 0.94 / 0.88, but A = 16 0.87 / 0.86 / 0.84 -> 0.85 / 0.84 / 0.79, so only for the two narrow row widths
    // (the test hook forces it for any A).
    const bool rows_ok = T % (rlcs::kRetraceProbsThreads * rlcs::kRetraceProbsItems) == 0 &&
                         (rlcs_hooks::g_row_blocks > 0 || (vec_rows && (A == 4 || A == 8)));
    st = finish_params(p, kVariant, total, T, workspace, workspace_bytes, vec, false, 1, false, rows_ok ? 2 : 0);
    if (st != RLCS_OK) return st;
    return rlcs::launch_retrace_probs(p, truncs != nullptr, vec, vec_rows, static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess
               ? RLCS_OK : RLCS_ERR_CUDA;
}

int rlcs_td_lambda(const float* rewards, const float* values, const uint8_t* dones, const uint8_t* truncs,
                   const float* trunc_bootstrap, const float* bootstrap, float* returns, int64_t N, int64_t T,
                   float gamma, float lambda, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    ScanParams p = {};
    Ptrs ps;
    int64_t total;
    bool vec;
    if (!unit_interval(gamma) || !unit_interval(lambda)) return RLCS_ERR_ARG;
    ps.add_f32(rewards); ps.add_f32(values); ps.add_f32(returns);
    int st = backward_common(p, ps, dones, truncs, trunc_bootstrap, bootstrap, N, T, &total, &vec);
    if (st != RLCS_OK || total == 0) return st;
    if (!rewards || !values || !returns) return RLCS_ERR_NULL;
    p.f0 = rewards; p.f1 = values; p.out0 = returns;
    p.gamma = gamma; p.decay = gamma * lambda; p.aux = gamma * (1.f - lambda);
    const int variant = choose_variant(rlcs::kTdLambda, truncs != nullptr, total, T);
    st = finish_params(p, variant, total, T, workspace, workspace_bytes, vec);
    if (st != RLCS_OK) return st;
    return run(rlcs::launch_td_lambda, p, variant, truncs != nullptr, vec, cuda_stream);
}

int rlcs_discounted_return(const float* rewards, const uint8_t* dones, const uint8_t* truncs,
                           const float* trunc_bootstrap, const float* bootstrap, float* returns, int64_t N,
                           int64_t T, float gamma, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    ScanParams p = {};
    Ptrs ps;
    int64_t total;
    bool vec;
    if (!unit_interval(gamma)) return RLCS_ERR_ARG;
    ps.add_f32(rewards); ps.add_f32(returns);
    int st = backward_common(p, ps, dones, truncs, trunc_bootstrap, bootstrap, N, T, &total, &vec);
    if (st != RLCS_OK || total == 0) return st;
    if (!rewards || !returns) return RLCS_ERR_NULL;
    p.f0 = rewards; p.out0 = returns;
    p.gamma = gamma; p.decay = gamma;
    const int variant = choose_variant(rlcs::kDisc, truncs != nullptr, total, T);
    st = finish_params(p, variant, total, T, workspace, workspace_bytes, vec);
    if (st != RLCS_OK) return st;
    return run(rlcs::launch_disc, p, variant, truncs != nullptr, vec, cuda_stream);
}

static int forward_scan(rlcs::Algo algo, const float* x, const uint8_t* dones, float* out, int64_t N, int64_t T,
                        float decay, int starts_at, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    ScanParams p = {};
    Ptrs ps;
    int64_t total;
    bool vec;
    int st = check_sizes(N, T, &total);
    if (st != RLCS_OK || total == 0) return st;
    if (!x || !dones || !out) return RLCS_ERR_NULL;
    ps.add_f32(x); ps.add_f32(out); ps.add_u8(dones);
    st = check_alignment(ps, &vec);
    if (st != RLCS_OK) return st;
    p.f0 = x; p.dones = dones; p.out0 = out; p.decay = decay; p.starts_at = starts_at != 0;
    const int variant = choose_variant(algo, false, total, T);
    st = finish_params(p, variant, total, T, workspace, workspace_bytes, vec);
    if (st != RLCS_OK) return st;
    return run(algo == rlcs::kElig ? rlcs::launch_elig : rlcs::launch_prefix, p, variant, false, vec, cuda_stream);
}

int rlcs_elig_trace(const float* x, const uint8_t* dones, float* traces, int64_t N, int64_t T, float gamma,
                    float lambda, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (!unit_interval(gamma) || !unit_interval(lambda)) return RLCS_ERR_ARG;
    return forward_scan(rlcs::kElig, x, dones, traces, N, T, gamma * lambda, 0, workspace, workspace_bytes, cuda_stream);
}

int rlcs_episodic_prefix_sum(const float* x, const uint8_t* dones, float* sums, int64_t N, int64_t T,
                             int starts_at, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return forward_scan(rlcs::kPrefix, x, dones, sums, N, T, 1.f, starts_at, workspace, workspace_bytes, cuda_stream);
}

int rlcs_affine_scan(const float* alpha, const float* beta, float* out, int64_t N, int64_t T, int forward,
                     void* workspace, size_t workspace_bytes, void* cuda_stream) {
    ScanParams p = {};
    Ptrs ps;
    int64_t total;
    bool vec;
    int st = check_sizes(N, T, &total);
    if (st != RLCS_OK || total == 0) return st;
    if (!alpha || !beta || !out) return RLCS_ERR_NULL;
    ps.add_f32(alpha); ps.add_f32(beta); ps.add_f32(out);
    st = check_alignment(ps, &vec);
    if (st != RLCS_OK) return st;
    p.f0 = alpha; p.f1 = beta; p.out0 = out;
    const int variant = choose_variant(forward ? rlcs::kAffineFwd : rlcs::kAffineBwd, false, total, T);
    st = finish_params(p, variant, total, T, workspace, workspace_bytes, vec);
    if (st != RLCS_OK) return st;
    return run(forward ? rlcs::launch_affine_fwd : rlcs::launch_affine_bwd, p, variant, false, vec, cuda_stream);
}

int rlcs_debug_set_tile_variant(int variant) {
    if (variant < -1 || variant >= rlcs::kNumVariants) return RLCS_ERR_ARG;
    // not compiled into either build (shape 21 exists in the bfloat16 build only; the fp32 entry points ignore it)
    if (variant >= 0 && !rlcs::variant_built(variant) && variant != 21) return RLCS_ERR_ARG;
    g_variant = variant;
    return RLCS_OK;
}

int rlcs_debug_variant_built(int variant) {
    return variant >= 0 && variant < rlcs::kNumVariants && rlcs::variant_built(variant) ? 1 : 0;
}

int rlcs_debug_tile_elems(int variant) {
    if (variant < 0 || variant >= rlcs::kNumVariants) return 0;
    return tile_elems(variant);
}

int rlcs_debug_variant_for(int algorithm, int has_truncs, int64_t N, int64_t T) {
    int64_t total = 0;
    if (algorithm < 0 || algorithm > rlcs::kAffineFwd || check_sizes(N, T, &total) != RLCS_OK || total == 0) return -1;
    return choose_variant(algorithm, has_truncs != 0, total, T);
}

int rlcs_debug_variant_info(int variant, int* threads, int* steps_per_thread, int* blocks_per_sm, int* ring_stages) {
    if (variant < 0 || variant >= rlcs::kNumVariants) return RLCS_ERR_ARG;
    const rlcs::TileVariant tv = rlcs::kVariants[variant];
    if (threads) *threads = tv.threads;
    if (steps_per_thread) *steps_per_thread = tv.items;
    if (blocks_per_sm) *blocks_per_sm = tv.min_blocks;
    if (ring_stages) *ring_stages = tv.stages;
    return RLCS_OK;
}

int rlcs_debug_set_row_blocks(int mode) {
    rlcs_hooks::g_row_blocks = mode;
    return RLCS_OK;
}

int rlcs_debug_allow_row_tiles(int on) {
    rlcs_hooks::g_row_tiles = on != 0;
    return RLCS_OK;
}

int rlcs_debug_set_dependent_launch(int on) {
    rlcs_hooks::g_pdl = on != 0;
    return RLCS_OK;
}

int rlcs_debug_allow_cluster_carry(int on) {
    g_cluster = on != 0;
    return RLCS_OK;
}

int rlcs_debug_force_wide_index(int on) {
    g_wide_index = on != 0;
    return RLCS_OK;
}

int rlcs_debug_set_carry_fault(int64_t mute_tile, int64_t spin_cap) {
    g_mute_tile = mute_tile;
    g_spin_cap = spin_cap;
    return RLCS_OK;
}

}  // extern "C"
