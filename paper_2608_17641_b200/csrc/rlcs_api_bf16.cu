// C ABI of the bfloat16-tensor entry points: the seven algorithms with every float tensor stored
// as bfloat16 (inputs, bootstrap values and outputs), arithmetic in fp32 on chip.  Same validation,
// tiling and carry machinery as the fp32 entry points; the kernels are the bfloat16 build of the
// same source (namespace rlcs_bf16).
#define RLCS_IO_BF16 1
#include "rlcs_host.cuh"

namespace {

namespace K = rlcs_bf16;

inline const io_t* in(const uint16_t* p) { return reinterpret_cast<const io_t*>(p); }
inline io_t* out(uint16_t* p) { return reinterpret_cast<io_t*>(p); }

// shared front half of the two forward entry points
int forward_common(ScanParams& p, Ptrs& ps, const uint16_t* x, const uint8_t* dones, uint16_t* y, int64_t N, int64_t T,
                   int64_t* total, bool* vec) {
    int st = check_sizes(N, T, total);
    if (st != RLCS_OK || *total == 0) return st;
    if (!x || !dones || !y) return RLCS_ERR_NULL;
    ps.add_f32(x); ps.add_f32(y); ps.add_u8(dones);
    st = check_alignment(ps, vec);
    if (st != RLCS_OK) return st;
    p.f0 = in(x); p.dones = dones; p.out0 = out(y);
    return RLCS_OK;
}

}  // namespace

extern "C" {

int rlcs_gae_bf16(const uint16_t* rewards, const uint16_t* values, const uint8_t* dones, const uint8_t* truncs,
                  const uint16_t* trunc_bootstrap, const uint16_t* bootstrap, uint16_t* advantages, uint16_t* returns,
                  int64_t N, int64_t T, float gamma, float lambda, void* workspace, size_t workspace_bytes,
                  void* cuda_stream) {
    ScanParams p = {};
    Ptrs ps;
    int64_t total;
    bool vec;
    if (!unit_interval(gamma) || !unit_interval(lambda)) return RLCS_ERR_ARG;
    ps.add_f32(rewards); ps.add_f32(values); ps.add_f32(advantages); ps.add_f32(returns);
    int st = backward_common(p, ps, dones, truncs, in(trunc_bootstrap), in(bootstrap), N, T, &total, &vec);
    if (st != RLCS_OK || total == 0) return st;
    if (!rewards || !values || !advantages) return RLCS_ERR_NULL;
    p.f0 = in(rewards); p.f1 = in(values); p.out0 = out(advantages); p.out1 = out(returns);
    p.gamma = gamma; p.decay = gamma * lambda;
    const int variant = choose_variant(K::kGae, truncs != nullptr, total, T);
    st = finish_params(p, variant, total, T, workspace, workspace_bytes, vec);
    if (st != RLCS_OK) return st;
    return run(K::launch_gae, p, variant, truncs != nullptr, vec, cuda_stream);
}

int rlcs_vtrace_bf16(const uint16_t* rewards, const uint16_t* values, const uint16_t* log_rhos, const uint8_t* dones,
                     const uint8_t* truncs, const uint16_t* trunc_bootstrap, const uint16_t* bootstrap, uint16_t* vs,
                     uint16_t* pg_advantages, int64_t N, int64_t T, float gamma, float rho_bar, float c_bar,
                     void* workspace, size_t workspace_bytes, void* cuda_stream) {
    ScanParams p = {};
    Ptrs ps;
    int64_t total;
    bool vec;
    if (!unit_interval(gamma) || !clip_ok(rho_bar) || !clip_ok(c_bar)) return RLCS_ERR_ARG;
    ps.add_f32(rewards); ps.add_f32(values); ps.add_f32(log_rhos); ps.add_f32(vs); ps.add_f32(pg_advantages);
    int st = backward_common(p, ps, dones, truncs, in(trunc_bootstrap), in(bootstrap), N, T, &total, &vec);
    if (st != RLCS_OK || total == 0) return st;
    if (!rewards || !values || !log_rhos || !vs) return RLCS_ERR_NULL;
    p.f0 = in(rewards); p.f1 = in(values); p.f3 = in(log_rhos); p.out0 = out(vs); p.out1 = out(pg_advantages);
    p.gamma = gamma; p.rho_bar = rho_bar; p.c_bar = c_bar;
    const int variant = choose_variant(K::kVtrace, truncs != nullptr, total, T);
    st = finish_params(p, variant, total, T, workspace, workspace_bytes, vec);
    if (st != RLCS_OK) return st;
    return run(K::launch_vtrace, p, variant, truncs != nullptr, vec, cuda_stream);
}

int rlcs_retrace_bf16(const uint16_t* rewards, const uint16_t* q_sa, const uint16_t* expected_q, const uint16_t* log_rhos,
                      const uint8_t* dones, const uint8_t* truncs, const uint16_t* trunc_bootstrap,
                      const uint16_t* bootstrap, uint16_t* q_targets, int64_t N, int64_t T, float gamma, float lambda,
                      float c_bar, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    ScanParams p = {};
    Ptrs ps;
    int64_t total;
    bool vec;
    if (!unit_interval(gamma) || !unit_interval(lambda) || !clip_ok(c_bar)) return RLCS_ERR_ARG;
    ps.add_f32(rewards); ps.add_f32(q_sa); ps.add_f32(expected_q); ps.add_f32(log_rhos); ps.add_f32(q_targets);
    int st = backward_common(p, ps, dones, truncs, in(trunc_bootstrap), in(bootstrap), N, T, &total, &vec);
    if (st != RLCS_OK || total == 0) return st;
    if (!rewards || !q_sa || !expected_q || !log_rhos || !q_targets) return RLCS_ERR_NULL;
    p.f0 = in(rewards); p.f1 = in(q_sa); p.f2 = in(expected_q); p.f3 = in(log_rhos); p.out0 = out(q_targets);
    p.gamma = gamma; p.aux = gamma * lambda; p.c_bar = c_bar;
    const int variant = choose_variant(K::kRetrace, truncs != nullptr, total, T);
    st = finish_params(p, variant, total, T, workspace, workspace_bytes, vec);
    if (st != RLCS_OK) return st;
    return run(K::launch_retrace, p, variant, truncs != nullptr, vec, cuda_stream);
}

int rlcs_td_lambda_bf16(const uint16_t* rewards, const uint16_t* values, const uint8_t* dones, const uint8_t* truncs,
                        const uint16_t* trunc_bootstrap, const uint16_t* bootstrap, uint16_t* returns, int64_t N,
                        int64_t T, float gamma, float lambda, void* workspace, size_t workspace_bytes,
                        void* cuda_stream) {
    ScanParams p = {};
    Ptrs ps;
    int64_t total;
    bool vec;
    if (!unit_interval(gamma) || !unit_interval(lambda)) return RLCS_ERR_ARG;
    ps.add_f32(rewards); ps.add_f32(values); ps.add_f32(returns);
    int st = backward_common(p, ps, dones, truncs, in(trunc_bootstrap), in(bootstrap), N, T, &total, &vec);
    if (st != RLCS_OK || total == 0) return st;
    if (!rewards || !values || !returns) return RLCS_ERR_NULL;
    p.f0 = in(rewards); p.f1 = in(values); p.out0 = out(returns);
    p.gamma = gamma; p.decay = gamma * lambda; p.aux = gamma * (1.f - lambda);
    const int variant = choose_variant(K::kTdLambda, truncs != nullptr, total, T);
    st = finish_params(p, variant, total, T, workspace, workspace_bytes, vec);
    if (st != RLCS_OK) return st;
    return run(K::launch_td_lambda, p, variant, truncs != nullptr, vec, cuda_stream);
}

int rlcs_discounted_return_bf16(const uint16_t* rewards, const uint8_t* dones, const uint8_t* truncs,
                                const uint16_t* trunc_bootstrap, const uint16_t* bootstrap, uint16_t* returns, int64_t N,
                                int64_t T, float gamma, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    ScanParams p = {};
    Ptrs ps;
    int64_t total;
    bool vec;
    if (!unit_interval(gamma)) return RLCS_ERR_ARG;
    ps.add_f32(rewards); ps.add_f32(returns);
    int st = backward_common(p, ps, dones, truncs, in(trunc_bootstrap), in(bootstrap), N, T, &total, &vec);
    if (st != RLCS_OK || total == 0) return st;
    if (!rewards || !returns) return RLCS_ERR_NULL;
    p.f0 = in(rewards); p.out0 = out(returns);
    p.gamma = gamma; p.decay = gamma;
    const int variant = choose_variant(K::kDisc, truncs != nullptr, total, T);
    st = finish_params(p, variant, total, T, workspace, workspace_bytes, vec);
    if (st != RLCS_OK) return st;
    return run(K::launch_disc, p, variant, truncs != nullptr, vec, cuda_stream);
}

int rlcs_elig_trace_bf16(const uint16_t* x, const uint8_t* dones, uint16_t* traces, int64_t N, int64_t T, float gamma,
                         float lambda, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    ScanParams p = {};
    Ptrs ps;
    int64_t total;
    bool vec;
    if (!unit_interval(gamma) || !unit_interval(lambda)) return RLCS_ERR_ARG;
    int st = forward_common(p, ps, x, dones, traces, N, T, &total, &vec);
    if (st != RLCS_OK || total == 0) return st;
    p.decay = gamma * lambda;
    const int variant = choose_variant(K::kElig, false, total, T);
    st = finish_params(p, variant, total, T, workspace, workspace_bytes, vec);
    if (st != RLCS_OK) return st;
    return run(K::launch_elig, p, variant, false, vec, cuda_stream);
}

int rlcs_episodic_prefix_sum_bf16(const uint16_t* x, const uint8_t* dones, uint16_t* sums, int64_t N, int64_t T,
                                  int starts_at, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    ScanParams p = {};
    Ptrs ps;
    int64_t total;
    bool vec;
    int st = forward_common(p, ps, x, dones, sums, N, T, &total, &vec);
    if (st != RLCS_OK || total == 0) return st;
    p.decay = 1.f;
    p.starts_at = starts_at != 0;
    const int variant = choose_variant(K::kPrefix, false, total, T);
    st = finish_params(p, variant, total, T, workspace, workspace_bytes, vec);
    if (st != RLCS_OK) return st;
    return run(K::launch_prefix, p, variant, false, vec, cuda_stream);
}

}  // extern "C"
