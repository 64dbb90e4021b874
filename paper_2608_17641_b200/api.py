"""Call-by-name front end over the C-ABI binding, with the argument names of the paper's
``compute_*`` functions (Section 6.1): picks the entry point from dtype and layout, keeps one carry
workspace per (device, stream, shape) so that repeated calls allocate nothing, and accepts
``torch.bool`` masks.  Workspace sharing rule: calls that use the same cached workspace are those
issued on the same stream, which orders them; calls on different streams get different workspaces.
A caller that passes ``workspace=`` itself must keep the calls sharing it ordered on the GPU.  Argument marshalling only -- every step runs in the CUDA kernels, there is no CPU path.

    adv, ret = compute_gae(rewards, values, dones, truncateds, bootstrap_values, bootstrap,
                           gamma=0.99, lam=0.95)

float32 tensors go to the fp32 entry points, bfloat16 tensors to the ``*_bf16`` ones (row-major
only); ``time_major=True`` takes ``[T, N]`` tensors (float32 only).  ``bootstrap_values`` is the
paper's 2-D tensor of continuation values at truncated steps, ``bootstrap`` its 1-D window-edge
vector (Section 4.2).
"""
from __future__ import annotations

from . import binding as _B

_workspaces: dict = {}


def _torch():
    import torch
    return torch


def _mask(m):
    """bool masks are reinterpreted as uint8 (same storage), uint8 passes through."""
    if m is None:
        return None
    torch = _torch()
    return m.view(torch.uint8) if m.dtype == torch.bool else m


def _workspace(like, N: int, T: int, nbytes: int | None = None, stream=None):
    """One initialised workspace per (device, stream, N, T, size), reused by every later call on that
    shape and stream.  The stream is part of the key because two calls share carry records and a
    call counter in the workspace: only calls ordered on one stream may share one."""
    if not like.is_cuda:
        raise TypeError("rlcs takes CUDA tensors (device pointers); there is no CPU path")
    s = _torch().cuda.current_stream(like.device) if stream is None else stream
    key = (like.device, int(s.cuda_stream), N, T, nbytes)
    ws = _workspaces.get(key)
    if ws is None:
        ws = _B.Workspace(N, T, device=like.device, stream=s, nbytes=nbytes)
        _workspaces[key] = ws
    return ws


def _kind(t, time_major: bool) -> str:
    torch = _torch()
    if t.dtype == torch.float32:
        return "tm" if time_major else "f32"
    if t.dtype == torch.bfloat16:
        if time_major:
            raise ValueError("time_major=True takes float32 tensors (the bfloat16 entry points are row-major)")
        return "bf16"
    raise TypeError(f"expected float32 or bfloat16 tensors, got {t.dtype}")


def _shape(t, time_major: bool):
    if t.dim() != 2:
        raise ValueError("expected 2-D [num_envs, seq_len] tensors ([seq_len, num_envs] with time_major=True)")
    return (t.shape[1], t.shape[0]) if time_major else (t.shape[0], t.shape[1])


def _ws_for(kind: str, like, N: int, T: int, workspace, stream=None):
    if workspace is not None:
        return workspace
    if kind == "tm":
        nbytes = int(_B.lib().rlcs_time_major_workspace_bytes(N, T))
        return _workspace(like, N, T, max(nbytes, 256), stream=stream) if nbytes else None
    return _workspace(like, N, T, stream=stream)


def compute_gae(rewards, values, dones, truncateds=None, bootstrap_values=None, bootstrap=None, *, gamma=0.99,
                lam=0.95, time_major=False, normalize=False, eps=1e-8, skip_mask=None, workspace=None, stream=None):
    """GAE advantages and returns (Section 3.3.1).  ``normalize``: advantages standardised over the
    whole batch (returns from the raw advantages).  ``skip_mask``: observation-skip masking (masked
    steps are transparent); returns (advantages, returns, filled values) then."""
    kind = _kind(rewards, time_major)
    N, T = _shape(rewards, time_major)
    dones, truncateds, skip_mask = _mask(dones), _mask(truncateds), _mask(skip_mask)
    if normalize or skip_mask is not None:
        if kind != "f32" or (normalize and skip_mask is not None):
            raise ValueError("normalize / skip_mask take row-major float32 tensors, one of the two at a time")
    if normalize:
        ws = workspace if workspace is not None else _workspace(
            rewards, N, T, int(_B.lib().rlcs_gae_normalized_workspace_bytes(N, T)), stream=stream)
        return _B.rlcs_gae_normalized(rewards, values, dones, truncateds, bootstrap_values, bootstrap, gamma=gamma, lam=lam,
                                      eps=eps, workspace=ws, stream=stream)
    ws = _ws_for(kind, rewards, N, T, workspace, stream)
    if skip_mask is not None:
        return _B.rlcs_gae_skip(rewards, values, dones, truncateds, bootstrap_values, bootstrap, skip=skip_mask, gamma=gamma,
                                lam=lam, workspace=ws, stream=stream)
    fn = {"f32": _B.rlcs_gae, "bf16": _B.rlcs_gae_bf16, "tm": _B.rlcs_gae_time_major}[kind]
    return fn(rewards, values, dones, truncateds, bootstrap_values, bootstrap, gamma=gamma, lam=lam, workspace=ws, stream=stream)


def compute_vtrace(rewards, values, log_rhos, dones, truncateds=None, bootstrap_values=None, bootstrap=None, *, gamma=0.99,
                   rho_bar=1.0, c_bar=1.0, time_major=False, workspace=None, stream=None):
    """V-Trace targets and policy-gradient advantages (Section 3.3.2); ``log_rhos = log pi - log mu``."""
    kind = _kind(rewards, time_major)
    N, T = _shape(rewards, time_major)
    fn = {"f32": _B.rlcs_vtrace, "bf16": _B.rlcs_vtrace_bf16, "tm": _B.rlcs_vtrace_time_major}[kind]
    return fn(rewards, values, log_rhos, _mask(dones), _mask(truncateds), bootstrap_values, bootstrap, gamma=gamma,
              rho_bar=rho_bar, c_bar=c_bar, workspace=_ws_for(kind, rewards, N, T, workspace, stream), stream=stream)


def compute_retrace(rewards, q_sa, expected_q, log_rhos, dones, truncateds=None, bootstrap_values=None, bootstrap=None, *,
                    gamma=0.99, lam=0.95, c_bar=1.0, time_major=False, workspace=None, stream=None):
    """Retrace(lambda) targets from per-step scalars (Section 3.3.3): Q(s_t,a_t), E_pi Q(s_t,.), log pi/mu."""
    kind = _kind(rewards, time_major)
    N, T = _shape(rewards, time_major)
    fn = {"f32": _B.rlcs_retrace, "bf16": _B.rlcs_retrace_bf16, "tm": _B.rlcs_retrace_time_major}[kind]
    return fn(rewards, q_sa, expected_q, log_rhos, _mask(dones), _mask(truncateds), bootstrap_values, bootstrap, gamma=gamma,
              lam=lam, c_bar=c_bar, workspace=_ws_for(kind, rewards, N, T, workspace, stream), stream=stream)


def compute_retrace_from_probs(rewards, q_values, target_probs, behaviour_probs, actions, dones, truncateds=None,
                               bootstrap_values=None, bootstrap=None, *, gamma=0.99, lam=0.95, c_bar=1.0, workspace=None,
                               stream=None):
    """Retrace(lambda) from the [N, T, A] Q-values and action probabilities (Section 7.3's input form)."""
    N, T = rewards.shape
    return _B.rlcs_retrace_probs(rewards, q_values, target_probs, behaviour_probs, actions, _mask(dones), _mask(truncateds),
                                 bootstrap_values, bootstrap, gamma=gamma, lam=lam, c_bar=c_bar,
                                 workspace=workspace if workspace is not None else _workspace(rewards, N, T, stream=stream),
                                 stream=stream)


def compute_td_lambda_returns(rewards, values, dones, truncateds=None, bootstrap_values=None, bootstrap=None, *, gamma=0.99,
                              lam=0.95, time_major=False, workspace=None, stream=None):
    """TD(lambda) returns (Section 3.3.4)."""
    kind = _kind(rewards, time_major)
    N, T = _shape(rewards, time_major)
    fn = {"f32": _B.rlcs_td_lambda, "bf16": _B.rlcs_td_lambda_bf16, "tm": _B.rlcs_td_lambda_time_major}[kind]
    return fn(rewards, values, _mask(dones), _mask(truncateds), bootstrap_values, bootstrap, gamma=gamma, lam=lam,
              workspace=_ws_for(kind, rewards, N, T, workspace, stream), stream=stream)


def compute_discounted_returns(rewards, dones, truncateds=None, bootstrap_values=None, bootstrap=None, *, gamma=0.99,
                               time_major=False, workspace=None, stream=None):
    """Discounted returns (Section 3.3.4, lambda = 1 without a value function)."""
    kind = _kind(rewards, time_major)
    N, T = _shape(rewards, time_major)
    fn = {"f32": _B.rlcs_discounted_return, "bf16": _B.rlcs_discounted_return_bf16,
          "tm": _B.rlcs_discounted_return_time_major}[kind]
    return fn(rewards, _mask(dones), _mask(truncateds), bootstrap_values, bootstrap, gamma=gamma,
              workspace=_ws_for(kind, rewards, N, T, workspace, stream), stream=stream)


def compute_eligibility_traces(x, dones, *, gamma=0.99, lam=0.95, beta=None, time_major=False, workspace=None, stream=None):
    """Eligibility traces (Section 3.3.5).  x [N, T]: scalar traces; x [N, T, D]: vector traces with the
    shared decay gamma*lam, or with a decay per component and step when ``beta`` [N, T, D] is given."""
    if x.dim() == 3:
        if time_major:
            raise ValueError("vector traces take [N, T, D] tensors")
        N, T, D = x.shape
        query = _B.lib().rlcs_elig_trace_vec_workspace_bytes if beta is None else _B.lib().rlcs_elig_trace_vec_beta_workspace_bytes
        nbytes = int(query(N, T, D))
        if workspace is None and nbytes:                       # few long rows: chunk records, cached like the others
            workspace = _workspace(x, N, T, nbytes, stream=stream)
        if beta is not None:
            return _B.rlcs_elig_trace_vec_beta(x, beta, _mask(dones), workspace=workspace, stream=stream)
        return _B.rlcs_elig_trace_vec(x, _mask(dones), gamma=gamma, lam=lam, workspace=workspace, stream=stream)
    if beta is not None:
        raise ValueError("beta goes with [N, T, D] vector traces")
    kind = _kind(x, time_major)
    N, T = _shape(x, time_major)
    fn = {"f32": _B.rlcs_elig_trace, "bf16": _B.rlcs_elig_trace_bf16, "tm": _B.rlcs_elig_trace_time_major}[kind]
    return fn(x, _mask(dones), gamma=gamma, lam=lam, workspace=_ws_for(kind, x, N, T, workspace, stream), stream=stream)


def compute_episodic_prefix_sum(x, dones, *, boundary="ends_at", time_major=False, workspace=None, stream=None):
    """Episodic prefix sums (Section 3.3.6); boundary = "ends_at" (dones marks last steps) or "starts_at"."""
    if boundary not in ("ends_at", "starts_at"):
        raise ValueError('boundary must be "ends_at" or "starts_at"')
    kind = _kind(x, time_major)
    N, T = _shape(x, time_major)
    fn = {"f32": _B.rlcs_episodic_prefix_sum, "bf16": _B.rlcs_episodic_prefix_sum_bf16,
          "tm": _B.rlcs_episodic_prefix_sum_time_major}[kind]
    return fn(x, _mask(dones), starts_at=(boundary == "starts_at"), workspace=_ws_for(kind, x, N, T, workspace, stream), stream=stream)
