"""ctypes binding of ``librlcs.so``: same names as the C ABI, argument marshalling only.

Every function takes CUDA ``torch.Tensor`` arguments (fp32 / uint8 / bool, contiguous), passes their
device pointers and the current CUDA stream to the C entry point and returns the output tensors.
Nothing is computed here; there is no CPU path.  A missing library raises at first use.
"""
from __future__ import annotations

import ctypes
import os
import threading

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "librlcs.so")

RLCS_OK = 0
RLCS_ERR_NULL, RLCS_ERR_SIZE, RLCS_ERR_ARG, RLCS_ERR_ALIGN = 1, 2, 3, 4
RLCS_ERR_WORKSPACE, RLCS_ERR_CUDA, RLCS_ERR_TIMEOUT, RLCS_ERR_LIMIT, RLCS_ERR_CAPTURE = 5, 6, 7, 8, 9

_vp, _i64, _f, _sz, _int = ctypes.c_void_p, ctypes.c_int64, ctypes.c_float, ctypes.c_size_t, ctypes.c_int
_TAIL = [_vp, _sz, _vp]          # workspace, workspace_bytes, cuda_stream

# name -> argtypes, exactly the declarations of include/rlcs.h
SIGNATURES = {
    "rlcs_status_string": ([_int], ctypes.c_char_p),
    "rlcs_workspace_bytes": ([_i64, _i64], _sz),
    "rlcs_workspace_init": ([_vp, _sz, _vp], _int),
    "rlcs_last_device_status": ([_vp, _vp], _int),
    "rlcs_gae": ([_vp] * 8 + [_i64, _i64, _f, _f] + _TAIL, _int),
    "rlcs_gae_normalized": ([_vp] * 8 + [_i64, _i64, _f, _f, _f, _int] + _TAIL, _int),
    "rlcs_gae_normalized_workspace_bytes": ([_i64, _i64], _sz),
    "rlcs_vtrace": ([_vp] * 9 + [_i64, _i64, _f, _f, _f] + _TAIL, _int),
    "rlcs_retrace": ([_vp] * 9 + [_i64, _i64, _f, _f, _f] + _TAIL, _int),
    "rlcs_retrace_probs": ([_vp] * 10 + [_i64, _i64, _i64, _f, _f, _f] + _TAIL, _int),
    "rlcs_td_lambda": ([_vp] * 7 + [_i64, _i64, _f, _f] + _TAIL, _int),
    "rlcs_discounted_return": ([_vp] * 6 + [_i64, _i64, _f] + _TAIL, _int),
    "rlcs_elig_trace": ([_vp] * 3 + [_i64, _i64, _f, _f] + _TAIL, _int),
    "rlcs_elig_trace_vec": ([_vp] * 3 + [_i64, _i64, _i64, _f, _f] + _TAIL, _int),
    "rlcs_elig_trace_vec_workspace_bytes": ([_i64, _i64, _i64], _sz),
    "rlcs_elig_trace_vec_beta": ([_vp] * 4 + [_i64, _i64, _i64] + _TAIL, _int),
    "rlcs_elig_trace_vec_beta_workspace_bytes": ([_i64, _i64, _i64], _sz),
    "rlcs_episodic_prefix_sum": ([_vp] * 3 + [_i64, _i64, _int] + _TAIL, _int),
    "rlcs_gae_skip": ([_vp] * 10 + [_i64, _i64, _f, _f] + _TAIL, _int),
    "rlcs_gae_no_alloc": ([_vp] * 8 + [_i64, _i64, _f, _f, _vp], _int),
    "rlcs_no_alloc_scratch_bytes": ([], _sz),
    "rlcs_no_alloc_last_device_status": ([_vp], _int),
    "rlcs_gae_carry_bytes": ([_i64, _i64, _int, _int], _sz),
    "rlcs_time_major_workspace_bytes": ([_i64, _i64], _sz),
    "rlcs_gae_time_major": ([_vp] * 8 + [_i64, _i64, _f, _f] + _TAIL, _int),
    "rlcs_vtrace_time_major": ([_vp] * 9 + [_i64, _i64, _f, _f, _f] + _TAIL, _int),
    "rlcs_retrace_time_major": ([_vp] * 9 + [_i64, _i64, _f, _f, _f] + _TAIL, _int),
    "rlcs_td_lambda_time_major": ([_vp] * 7 + [_i64, _i64, _f, _f] + _TAIL, _int),
    "rlcs_discounted_return_time_major": ([_vp] * 6 + [_i64, _i64, _f] + _TAIL, _int),
    "rlcs_elig_trace_time_major": ([_vp] * 3 + [_i64, _i64, _f, _f] + _TAIL, _int),
    "rlcs_episodic_prefix_sum_time_major": ([_vp] * 3 + [_i64, _i64, _int] + _TAIL, _int),
    "rlcs_gae_bf16": ([_vp] * 8 + [_i64, _i64, _f, _f] + _TAIL, _int),
    "rlcs_vtrace_bf16": ([_vp] * 9 + [_i64, _i64, _f, _f, _f] + _TAIL, _int),
    "rlcs_retrace_bf16": ([_vp] * 9 + [_i64, _i64, _f, _f, _f] + _TAIL, _int),
    "rlcs_td_lambda_bf16": ([_vp] * 7 + [_i64, _i64, _f, _f] + _TAIL, _int),
    "rlcs_discounted_return_bf16": ([_vp] * 6 + [_i64, _i64, _f] + _TAIL, _int),
    "rlcs_elig_trace_bf16": ([_vp] * 3 + [_i64, _i64, _f, _f] + _TAIL, _int),
    "rlcs_episodic_prefix_sum_bf16": ([_vp] * 3 + [_i64, _i64, _int] + _TAIL, _int),
    "rlcs_affine_scan": ([_vp] * 3 + [_i64, _i64, _int] + _TAIL, _int),
    "rlcs_debug_set_tile_variant": ([_int], _int),
    "rlcs_debug_tile_elems": ([_int], _int),
    "rlcs_debug_set_carry_fault": ([_i64, _i64], _int),
    "rlcs_debug_time_major_path": ([_int], None),
    "rlcs_debug_vec_trace_plan": ([_int, _int], None),
    "rlcs_debug_stream_copy": ([_vp, _vp, _sz, _sz, _vp], _int),
    "rlcs_debug_force_wide_index": ([_int], _int),
    "rlcs_debug_allow_cluster_carry": ([_int], _int),
    "rlcs_debug_set_dependent_launch": ([_int], _int),
    "rlcs_debug_allow_row_tiles": ([_int], _int),
    "rlcs_debug_set_row_blocks": ([_int], _int),
    "rlcs_debug_variant_for": ([_int, _int, _i64, _i64], _int),
    "rlcs_debug_variant_built": ([_int], _int),
    "rlcs_debug_variant_info": ([_int] + [ctypes.POINTER(ctypes.c_int)] * 4, _int),
}

_lib = None
_lock = threading.Lock()


class RlcsError(RuntimeError):
    def __init__(self, status: int):
        self.status = status
        super().__init__(lib().rlcs_status_string(status).decode())


_recording = threading.local()        # .calls: list while prepare() runs a wrapper, absent otherwise


class _Recorder:
    """Stands in for the library while prepare() runs a wrapper: records (C function, arguments) of
    every compute call instead of making it; anything else (size queries, ...) goes to the library."""

    def __init__(self, real):
        self._real = real

    def __getattr__(self, name):
        fn = getattr(self._real, name)
        compute = (fn.restype is _int and fn.argtypes and fn.argtypes[-1] is _vp and not name.startswith("rlcs_debug")
                   and name not in ("rlcs_workspace_init", "rlcs_last_device_status", "rlcs_no_alloc_last_device_status"))
        if not compute:
            return fn

        def record(*args):
            _recording.calls.append((fn, args))
            return RLCS_OK
        return record


class Prepared:
    """A call whose arguments were checked and marshalled once (prepare()).  Calling it only makes the
    C call(s) -- a few microseconds of host time instead of the 12-28 that dtype, shape, device and
    pointer marshalling cost per call -- on the current stream, or on `stream_handle` (a raw
    cudaStream_t as int) when given.  The tensors are kept alive by this object; `outputs` is what the
    wrapper would have returned.  The caller must not free or resize them while it is in use, and must
    call it with the device current on which it was prepared."""

    def __init__(self, calls, outputs, keep):
        self._calls, self.outputs, self._keep = calls, outputs, keep

    def __call__(self, stream_handle=None):
        h = _stream() if stream_handle is None else stream_handle
        for fn, args in self._calls:
            st = fn(*args[:-1], h)
            if st != RLCS_OK:
                raise RlcsError(st)
        return self.outputs


def prepare(wrapper, *args, **kwargs) -> Prepared:
    """Run one of this module's rlcs_* wrappers in recording mode: all of its checks happen now,
    outputs and workspace are allocated (and the workspace initialised) now -- pass them in to control
    that -- and no kernel is launched.  Not thread-safe: no other thread may use this module meanwhile.
    The returned object repeats the call at C-call cost, e.g. inside a training loop on fixed buffers:

        step = prepare(rlcs_gae, rewards, values, dones, gamma=0.99, lam=0.95, workspace=ws)
        ...
        adv, ret = step()
    """
    real = lib()
    global _lib
    _recording.calls = []
    with _lock:
        _lib = _Recorder(real)
    try:
        outputs = wrapper(*args, **kwargs)
        calls = list(_recording.calls)
    finally:
        with _lock:
            _lib = real
        del _recording.calls
    if not calls:
        raise ValueError("prepare() takes one of the rlcs_* compute wrappers of this module")
    return Prepared(calls, outputs, (args, kwargs))


def lib() -> ctypes.CDLL:
    """The loaded C library (loaded once).  Raises if it has not been built."""
    global _lib
    with _lock:
        if _lib is None:
            if not os.path.exists(LIB_PATH):
                raise RuntimeError(
                    f"{LIB_PATH} is missing: build it with `python -m paper_2608_17641_b200.build` "
                    "(there is no fallback path)")
            L = ctypes.CDLL(LIB_PATH)
            for name, (argtypes, restype) in SIGNATURES.items():
                fn = getattr(L, name)
                fn.argtypes = argtypes
                fn.restype = restype
            _lib = L
    return _lib


def _check(status: int):
    if status != RLCS_OK:
        raise RlcsError(status)


def _torch():
    import torch
    return torch


_cuda_current_device = None


def _current_device() -> int:
    global _cuda_current_device
    if _cuda_current_device is None:
        _cuda_current_device = _torch().cuda.current_device
    return _cuda_current_device()


def _require_current_device(t, what: str = "tensor"):
    """The library launches on the current device and the current stream of that device: a tensor
    (or workspace) that lives on another GPU would hand the kernel a pointer it must not touch."""
    index, cur = t.get_device(), _current_device()
    if index is not None and index >= 0 and index != cur:
        raise ValueError(f"{what} is on cuda:{index} but the current device is cuda:{cur}; "
                         f"call under torch.cuda.device({index})")


def _ptr(t, dtype_kind: str, shape=None):
    """Device pointer of a tensor (None -> NULL) after dtype / device / layout checks."""
    if t is None:
        return None
    torch = _torch()
    if not t.is_cuda:
        raise TypeError("rlcs takes CUDA tensors (device pointers); there is no CPU path")
    _require_current_device(t)
    if dtype_kind == "f32":
        if t.dtype != torch.float32:
            raise TypeError(f"expected float32, got {t.dtype}")     # the method is fp32-only
    elif dtype_kind == "bf16":
        if t.dtype != torch.bfloat16:
            raise TypeError(f"expected bfloat16, got {t.dtype}")
    elif t.dtype not in (torch.uint8, torch.bool):
        raise TypeError(f"expected a uint8/bool mask, got {t.dtype}")
    if not t.is_contiguous():
        raise ValueError("rlcs takes contiguous row-major tensors")
    if shape is not None and tuple(t.shape) != tuple(shape):
        raise ValueError(f"expected shape {tuple(shape)}, got {tuple(t.shape)}")
    return t.data_ptr()


def _alloc(shape, dtype, device):
    """Device memory for outputs and workspaces the binding creates itself (torch's allocator).  A
    module-level function so that a test harness can substitute an allocator that adds guard bands."""
    return _torch().empty(shape, dtype=dtype, device=device)


def _stream(stream=None):
    torch = _torch()
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


class Workspace:
    """Caller-owned carry workspace (device memory held by a torch tensor), initialised once."""

    def __init__(self, N: int, T: int, device="cuda", stream=None, nbytes: int | None = None):
        torch = _torch()
        self.nbytes = int(lib().rlcs_workspace_bytes(N, T)) if nbytes is None else int(nbytes)
        self.buf = _alloc((max(self.nbytes, 16),), torch.uint8, device) if self.nbytes else None
        if self.buf is not None:
            if stream is not None:
                self.buf.record_stream(stream)     # the caching allocator must not hand it out again before that stream is done
            _check(lib().rlcs_workspace_init(self.buf.data_ptr(), self.nbytes, _stream(stream)))

    @property
    def ptr(self):
        return None if self.buf is None else self.buf.data_ptr()

    def device_status(self, stream=None) -> int:
        return lib().rlcs_last_device_status(self.ptr, _stream(stream))


def workspace_bytes(N: int, T: int) -> int:
    return int(lib().rlcs_workspace_bytes(N, T))


def _ws(ws: Workspace | None):
    if ws is None:
        return (None, 0)
    if ws.buf is not None:
        _require_current_device(ws.buf, "workspace")
    return (ws.ptr, ws.nbytes)


def _out(like, out):
    torch = _torch()
    return _alloc(tuple(like.shape), torch.float32, like.device) if out is None else out


def rlcs_gae(rewards, values, dones, truncs=None, trunc_bootstrap=None, bootstrap=None, *, gamma, lam,
             advantages=None, returns=None, want_returns=True, workspace=None, stream=None):
    N, T = rewards.shape
    adv = _out(rewards, advantages)
    ret = (_out(rewards, returns) if want_returns else None)
    wp, wb = _ws(workspace)
    _check(lib().rlcs_gae(_ptr(rewards, "f32"), _ptr(values, "f32", (N, T)), _ptr(dones, "u8", (N, T)),
                          _ptr(truncs, "u8", (N, T)), _ptr(trunc_bootstrap, "f32", (N, T)),
                          _ptr(bootstrap, "f32", (N,)), _ptr(adv, "f32", (N, T)), _ptr(ret, "f32", (N, T)),
                          N, T, gamma, lam, wp, wb, _stream(stream)))
    return (adv, ret) if want_returns else adv


def rlcs_gae_normalized(rewards, values, dones, truncs=None, trunc_bootstrap=None, bootstrap=None, *, gamma, lam,
                        eps=1e-8, ddof=1, advantages=None, returns=None, want_returns=True, workspace=None, stream=None):
    """GAE + advantage normalisation over all N*T steps.  `workspace` must be a Workspace created with
    nbytes=rlcs_gae_normalized_workspace_bytes(N, T) (one is made on the fly when omitted)."""
    N, T = rewards.shape
    adv = _out(rewards, advantages)
    ret = (_out(rewards, returns) if want_returns else None)
    if workspace is None:
        workspace = Workspace(N, T, device=rewards.device, stream=stream,
                              nbytes=int(lib().rlcs_gae_normalized_workspace_bytes(N, T)))
    wp, wb = _ws(workspace)
    _check(lib().rlcs_gae_normalized(_ptr(rewards, "f32"), _ptr(values, "f32", (N, T)), _ptr(dones, "u8", (N, T)),
                                     _ptr(truncs, "u8", (N, T)), _ptr(trunc_bootstrap, "f32", (N, T)),
                                     _ptr(bootstrap, "f32", (N,)), _ptr(adv, "f32", (N, T)), _ptr(ret, "f32", (N, T)),
                                     N, T, gamma, lam, eps, ddof, wp, wb, _stream(stream)))
    return (adv, ret) if want_returns else adv


def rlcs_gae_skip(rewards, values, dones, truncs=None, trunc_bootstrap=None, bootstrap=None, *, skip, gamma, lam,
                  values_filled=None, advantages=None, returns=None, want_returns=True, workspace=None, stream=None):
    """GAE with observation-skip masking (skip != 0: masked, transparent step).  Returns
    (advantages, returns = A + W, values_filled = W), or (advantages, values_filled) without returns."""
    N, T = rewards.shape
    fil = _out(rewards, values_filled)
    adv = _out(rewards, advantages)
    ret = (_out(rewards, returns) if want_returns else None)
    wp, wb = _ws(workspace)
    _check(lib().rlcs_gae_skip(_ptr(rewards, "f32"), _ptr(values, "f32", (N, T)), _ptr(dones, "u8", (N, T)),
                               _ptr(truncs, "u8", (N, T)), _ptr(trunc_bootstrap, "f32", (N, T)),
                               _ptr(bootstrap, "f32", (N,)), _ptr(skip, "u8", (N, T)), _ptr(fil, "f32", (N, T)),
                               _ptr(adv, "f32", (N, T)), _ptr(ret, "f32", (N, T)), N, T, gamma, lam, wp, wb,
                               _stream(stream)))
    return (adv, ret, fil) if want_returns else (adv, fil)


def rlcs_gae_no_alloc(rewards, values, dones, truncs=None, trunc_bootstrap=None, bootstrap=None, *, gamma, lam,
                      advantages=None, returns=None, want_returns=True, stream=None):
    """GAE through the entry point that takes no workspace: the carry scratch is a fixed device
    array inside the library, so this call path performs no device allocation (pass `advantages`
    and `returns` to keep torch from allocating the outputs either).  Calls must not overlap on
    the GPU; the first call on a device should happen outside stream capture."""
    N, T = rewards.shape
    adv = _out(rewards, advantages)
    ret = (_out(rewards, returns) if want_returns else None)
    _check(lib().rlcs_gae_no_alloc(_ptr(rewards, "f32"), _ptr(values, "f32", (N, T)), _ptr(dones, "u8", (N, T)),
                                   _ptr(truncs, "u8", (N, T)), _ptr(trunc_bootstrap, "f32", (N, T)),
                                   _ptr(bootstrap, "f32", (N,)), _ptr(adv, "f32", (N, T)), _ptr(ret, "f32", (N, T)),
                                   N, T, gamma, lam, _stream(stream)))
    return (adv, ret) if want_returns else adv


def rlcs_no_alloc_last_device_status(stream=None) -> int:
    """Device status of the rlcs_gae_no_alloc calls on the current device (synchronises the stream,
    clears the word): RLCS_OK or RLCS_ERR_TIMEOUT."""
    return int(lib().rlcs_no_alloc_last_device_status(_stream(stream)))


def rlcs_vtrace(rewards, values, log_rhos, dones, truncs=None, trunc_bootstrap=None, bootstrap=None, *,
                gamma, rho_bar=1.0, c_bar=1.0, vs=None, pg_advantages=None, want_advantages=True,
                workspace=None, stream=None):
    N, T = rewards.shape
    vs = _out(rewards, vs)
    adv = (_out(rewards, pg_advantages) if want_advantages else None)
    wp, wb = _ws(workspace)
    _check(lib().rlcs_vtrace(_ptr(rewards, "f32"), _ptr(values, "f32", (N, T)), _ptr(log_rhos, "f32", (N, T)),
                             _ptr(dones, "u8", (N, T)), _ptr(truncs, "u8", (N, T)),
                             _ptr(trunc_bootstrap, "f32", (N, T)), _ptr(bootstrap, "f32", (N,)),
                             _ptr(vs, "f32", (N, T)), _ptr(adv, "f32", (N, T)), N, T, gamma, rho_bar, c_bar,
                             wp, wb, _stream(stream)))
    return (vs, adv) if want_advantages else vs


def rlcs_retrace(rewards, q_sa, expected_q, log_rhos, dones, truncs=None, trunc_bootstrap=None,
                 bootstrap=None, *, gamma, lam, c_bar=1.0, q_targets=None, workspace=None, stream=None):
    N, T = rewards.shape
    out = _out(rewards, q_targets)
    wp, wb = _ws(workspace)
    _check(lib().rlcs_retrace(_ptr(rewards, "f32"), _ptr(q_sa, "f32", (N, T)), _ptr(expected_q, "f32", (N, T)),
                              _ptr(log_rhos, "f32", (N, T)), _ptr(dones, "u8", (N, T)), _ptr(truncs, "u8", (N, T)),
                              _ptr(trunc_bootstrap, "f32", (N, T)), _ptr(bootstrap, "f32", (N,)),
                              _ptr(out, "f32", (N, T)), N, T, gamma, lam, c_bar, wp, wb, _stream(stream)))
    return out


def rlcs_retrace_probs(rewards, q_values, target_probs, behaviour_probs, actions, dones, truncs=None,
                       trunc_bootstrap=None, bootstrap=None, *, gamma, lam, c_bar=1.0, q_targets=None, workspace=None,
                       stream=None):
    """Retrace(lambda) from [N,T,A] Q-values / target / behaviour probabilities and int32 actions [N,T]."""
    torch = _torch()
    N, T = rewards.shape
    A = q_values.shape[2]
    if actions.dtype != torch.int32 or not actions.is_cuda or not actions.is_contiguous() or tuple(actions.shape) != (N, T):
        raise TypeError("actions must be a contiguous CUDA int32 tensor of shape [N, T]")
    out = _out(rewards, q_targets)
    wp, wb = _ws(workspace)
    _check(lib().rlcs_retrace_probs(_ptr(rewards, "f32"), _ptr(q_values, "f32", (N, T, A)),
                                    _ptr(target_probs, "f32", (N, T, A)), _ptr(behaviour_probs, "f32", (N, T, A)),
                                    actions.data_ptr(), _ptr(dones, "u8", (N, T)), _ptr(truncs, "u8", (N, T)),
                                    _ptr(trunc_bootstrap, "f32", (N, T)), _ptr(bootstrap, "f32", (N,)),
                                    _ptr(out, "f32", (N, T)), N, T, A, gamma, lam, c_bar, wp, wb, _stream(stream)))
    return out


def rlcs_td_lambda(rewards, values, dones, truncs=None, trunc_bootstrap=None, bootstrap=None, *, gamma, lam,
                   returns=None, workspace=None, stream=None):
    N, T = rewards.shape
    out = _out(rewards, returns)
    wp, wb = _ws(workspace)
    _check(lib().rlcs_td_lambda(_ptr(rewards, "f32"), _ptr(values, "f32", (N, T)), _ptr(dones, "u8", (N, T)),
                                _ptr(truncs, "u8", (N, T)), _ptr(trunc_bootstrap, "f32", (N, T)),
                                _ptr(bootstrap, "f32", (N,)), _ptr(out, "f32", (N, T)), N, T, gamma, lam,
                                wp, wb, _stream(stream)))
    return out


def rlcs_discounted_return(rewards, dones, truncs=None, trunc_bootstrap=None, bootstrap=None, *, gamma,
                           returns=None, workspace=None, stream=None):
    N, T = rewards.shape
    out = _out(rewards, returns)
    wp, wb = _ws(workspace)
    _check(lib().rlcs_discounted_return(_ptr(rewards, "f32"), _ptr(dones, "u8", (N, T)), _ptr(truncs, "u8", (N, T)),
                                        _ptr(trunc_bootstrap, "f32", (N, T)), _ptr(bootstrap, "f32", (N,)),
                                        _ptr(out, "f32", (N, T)), N, T, gamma, wp, wb, _stream(stream)))
    return out


def rlcs_elig_trace(x, dones, *, gamma, lam, traces=None, workspace=None, stream=None):
    N, T = x.shape
    out = _out(x, traces)
    wp, wb = _ws(workspace)
    _check(lib().rlcs_elig_trace(_ptr(x, "f32"), _ptr(dones, "u8", (N, T)), _ptr(out, "f32", (N, T)), N, T,
                                 gamma, lam, wp, wb, _stream(stream)))
    return out


def rlcs_elig_trace_vec(x, dones, *, gamma, lam, traces=None, workspace=None, stream=None):
    """Vector-valued eligibility trace: x [N,T,D], dones [N,T].  A workspace is made on the fly when the
    time axis has to be cut and none is given."""
    N, T, D = x.shape
    out = _out(x, traces)
    if workspace is None:
        nbytes = int(lib().rlcs_elig_trace_vec_workspace_bytes(N, T, D))
        workspace = Workspace(N, T, device=x.device, stream=stream, nbytes=nbytes) if nbytes else None
    wp, wb = _ws(workspace)
    _check(lib().rlcs_elig_trace_vec(_ptr(x, "f32"), _ptr(dones, "u8", (N, T)), _ptr(out, "f32", (N, T, D)), N, T, D,
                                     gamma, lam, wp, wb, _stream(stream)))
    return out


def rlcs_elig_trace_vec_beta(x, beta, dones, *, traces=None, workspace=None, stream=None):
    """Eligibility trace with a decay per component and step: x, beta [N,T,D], dones [N,T]."""
    N, T, D = x.shape
    out = _out(x, traces)
    if workspace is None:
        nbytes = int(lib().rlcs_elig_trace_vec_beta_workspace_bytes(N, T, D))
        workspace = Workspace(N, T, device=x.device, stream=stream, nbytes=nbytes) if nbytes else None
    wp, wb = _ws(workspace)
    _check(lib().rlcs_elig_trace_vec_beta(_ptr(x, "f32"), _ptr(beta, "f32", (N, T, D)), _ptr(dones, "u8", (N, T)),
                                          _ptr(out, "f32", (N, T, D)), N, T, D, wp, wb, _stream(stream)))
    return out


def rlcs_episodic_prefix_sum(x, dones, *, starts_at=False, sums=None, workspace=None, stream=None):
    N, T = x.shape
    out = _out(x, sums)
    wp, wb = _ws(workspace)
    _check(lib().rlcs_episodic_prefix_sum(_ptr(x, "f32"), _ptr(dones, "u8", (N, T)), _ptr(out, "f32", (N, T)),
                                          N, T, int(bool(starts_at)), wp, wb, _stream(stream)))
    return out


def rlcs_affine_scan(alpha, beta, *, forward=False, out=None, workspace=None, stream=None):
    N, T = alpha.shape
    out = _out(alpha, out)
    wp, wb = _ws(workspace)
    _check(lib().rlcs_affine_scan(_ptr(alpha, "f32"), _ptr(beta, "f32", (N, T)), _ptr(out, "f32", (N, T)), N, T,
                                  int(bool(forward)), wp, wb, _stream(stream)))
    return out


def rlcs_debug_set_tile_variant(variant: int):
    _check(lib().rlcs_debug_set_tile_variant(variant))


def rlcs_debug_tile_elems(variant: int) -> int:
    return int(lib().rlcs_debug_tile_elems(variant))


ALGORITHM_IDS = {"gae": 0, "td_lambda": 1, "discounted_return": 2, "vtrace": 3, "retrace": 4, "elig_trace": 5,
                 "episodic_prefix_sum": 6}


def rlcs_debug_variant_for(algorithm: str, has_truncs: bool, N: int, T: int) -> dict:
    """The kernel variant a call would use, as {variant, threads, steps_per_thread, blocks_per_sm, ring_stages}."""
    v = int(lib().rlcs_debug_variant_for(ALGORITHM_IDS[algorithm], int(bool(has_truncs)), N, T))
    out = [ctypes.c_int() for _ in range(4)]
    _check(lib().rlcs_debug_variant_info(v, *[ctypes.byref(o) for o in out]))
    return dict(variant=v, threads=out[0].value, steps_per_thread=out[1].value, blocks_per_sm=out[2].value,
                ring_stages=out[3].value)


def rlcs_debug_set_row_blocks(mode: int = -1):
    """Test hook: one thread block per row: -1 = when there are enough rows (default), 0 = never, 1 = whenever legal."""
    _check(lib().rlcs_debug_set_row_blocks(int(mode)))


def rlcs_debug_allow_row_tiles(on: bool):
    """Test hook: allow (default) or forbid row-aligned tiling; without it short rows that do not divide the tile use the look-back."""
    _check(lib().rlcs_debug_allow_row_tiles(int(bool(on))))


def rlcs_debug_variant_built(variant: int) -> bool:
    """Whether that tile variant is compiled into the loaded library."""
    return bool(lib().rlcs_debug_variant_built(int(variant)))


def rlcs_debug_set_dependent_launch(on: bool):
    """Measurement hook: launch the row-major scan kernels with (default) or without programmatic stream serialisation."""
    _check(lib().rlcs_debug_set_dependent_launch(int(bool(on))))


def rlcs_debug_allow_cluster_carry(on: bool):
    _check(lib().rlcs_debug_allow_cluster_carry(int(bool(on))))


def rlcs_debug_force_wide_index(on: bool):
    _check(lib().rlcs_debug_force_wide_index(int(bool(on))))


def rlcs_debug_set_carry_fault(mute_tile: int = -1, spin_cap: int = 0):
    _check(lib().rlcs_debug_set_carry_fault(mute_tile, spin_cap))


def rlcs_debug_stream_copy(src, dst, read_bytes: int, write_bytes: int, stream=None):
    """Streaming read of read_bytes from src and write of write_bytes to dst (measurement hook)."""
    _check(lib().rlcs_debug_stream_copy(src.data_ptr(), dst.data_ptr(), int(read_bytes), int(write_bytes), _stream(stream)))


def rlcs_debug_vec_trace_plan(batch: int = 0, chunks: int = 0):
    """Test hook: force the load-ahead depth (8/16/32) and the number of time chunks of the vector traces."""
    lib().rlcs_debug_vec_trace_plan(int(batch), int(chunks))


def rlcs_debug_time_major_path(path: int = 0):
    """1 = register walk only; anything else = shared-memory ring wherever alignment allows (default)."""
    lib().rlcs_debug_time_major_path(int(path))


# ------------------------------------------------------------------------------------------ bfloat16 tensors
def _out16(like, out):
    torch = _torch()
    return _alloc(tuple(like.shape), torch.bfloat16, like.device) if out is None else out


def rlcs_gae_bf16(rewards, values, dones, truncs=None, trunc_bootstrap=None, bootstrap=None, *, gamma, lam,
                  advantages=None, returns=None, want_returns=True, workspace=None, stream=None):
    """GAE on bfloat16 tensors (fp32 arithmetic on chip, outputs rounded to bfloat16 on store)."""
    N, T = rewards.shape
    adv = _out16(rewards, advantages)
    ret = (_out16(rewards, returns) if want_returns else None)
    wp, wb = _ws(workspace)
    _check(lib().rlcs_gae_bf16(_ptr(rewards, "bf16"), _ptr(values, "bf16", (N, T)), _ptr(dones, "u8", (N, T)),
                               _ptr(truncs, "u8", (N, T)), _ptr(trunc_bootstrap, "bf16", (N, T)),
                               _ptr(bootstrap, "bf16", (N,)), _ptr(adv, "bf16", (N, T)), _ptr(ret, "bf16", (N, T)),
                               N, T, gamma, lam, wp, wb, _stream(stream)))
    return (adv, ret) if want_returns else adv


def rlcs_vtrace_bf16(rewards, values, log_rhos, dones, truncs=None, trunc_bootstrap=None, bootstrap=None, *,
                     gamma, rho_bar=1.0, c_bar=1.0, vs=None, pg_advantages=None, want_advantages=True,
                     workspace=None, stream=None):
    N, T = rewards.shape
    vs = _out16(rewards, vs)
    adv = (_out16(rewards, pg_advantages) if want_advantages else None)
    wp, wb = _ws(workspace)
    _check(lib().rlcs_vtrace_bf16(_ptr(rewards, "bf16"), _ptr(values, "bf16", (N, T)), _ptr(log_rhos, "bf16", (N, T)),
                                  _ptr(dones, "u8", (N, T)), _ptr(truncs, "u8", (N, T)),
                                  _ptr(trunc_bootstrap, "bf16", (N, T)), _ptr(bootstrap, "bf16", (N,)),
                                  _ptr(vs, "bf16", (N, T)), _ptr(adv, "bf16", (N, T)), N, T, gamma, rho_bar, c_bar,
                                  wp, wb, _stream(stream)))
    return (vs, adv) if want_advantages else vs


def rlcs_retrace_bf16(rewards, q_sa, expected_q, log_rhos, dones, truncs=None, trunc_bootstrap=None, bootstrap=None, *,
                      gamma, lam, c_bar=1.0, q_targets=None, workspace=None, stream=None):
    N, T = rewards.shape
    out = _out16(rewards, q_targets)
    wp, wb = _ws(workspace)
    _check(lib().rlcs_retrace_bf16(_ptr(rewards, "bf16"), _ptr(q_sa, "bf16", (N, T)), _ptr(expected_q, "bf16", (N, T)),
                                   _ptr(log_rhos, "bf16", (N, T)), _ptr(dones, "u8", (N, T)), _ptr(truncs, "u8", (N, T)),
                                   _ptr(trunc_bootstrap, "bf16", (N, T)), _ptr(bootstrap, "bf16", (N,)),
                                   _ptr(out, "bf16", (N, T)), N, T, gamma, lam, c_bar, wp, wb, _stream(stream)))
    return out


def rlcs_td_lambda_bf16(rewards, values, dones, truncs=None, trunc_bootstrap=None, bootstrap=None, *, gamma, lam,
                        returns=None, workspace=None, stream=None):
    N, T = rewards.shape
    out = _out16(rewards, returns)
    wp, wb = _ws(workspace)
    _check(lib().rlcs_td_lambda_bf16(_ptr(rewards, "bf16"), _ptr(values, "bf16", (N, T)), _ptr(dones, "u8", (N, T)),
                                     _ptr(truncs, "u8", (N, T)), _ptr(trunc_bootstrap, "bf16", (N, T)),
                                     _ptr(bootstrap, "bf16", (N,)), _ptr(out, "bf16", (N, T)), N, T, gamma, lam,
                                     wp, wb, _stream(stream)))
    return out


def rlcs_discounted_return_bf16(rewards, dones, truncs=None, trunc_bootstrap=None, bootstrap=None, *, gamma,
                                returns=None, workspace=None, stream=None):
    N, T = rewards.shape
    out = _out16(rewards, returns)
    wp, wb = _ws(workspace)
    _check(lib().rlcs_discounted_return_bf16(_ptr(rewards, "bf16"), _ptr(dones, "u8", (N, T)), _ptr(truncs, "u8", (N, T)),
                                             _ptr(trunc_bootstrap, "bf16", (N, T)), _ptr(bootstrap, "bf16", (N,)),
                                             _ptr(out, "bf16", (N, T)), N, T, gamma, wp, wb, _stream(stream)))
    return out


def rlcs_elig_trace_bf16(x, dones, *, gamma, lam, traces=None, workspace=None, stream=None):
    N, T = x.shape
    out = _out16(x, traces)
    wp, wb = _ws(workspace)
    _check(lib().rlcs_elig_trace_bf16(_ptr(x, "bf16"), _ptr(dones, "u8", (N, T)), _ptr(out, "bf16", (N, T)), N, T,
                                      gamma, lam, wp, wb, _stream(stream)))
    return out


def rlcs_episodic_prefix_sum_bf16(x, dones, *, starts_at=False, sums=None, workspace=None, stream=None):
    N, T = x.shape
    out = _out16(x, sums)
    wp, wb = _ws(workspace)
    _check(lib().rlcs_episodic_prefix_sum_bf16(_ptr(x, "bf16"), _ptr(dones, "u8", (N, T)), _ptr(out, "bf16", (N, T)),
                                               N, T, int(bool(starts_at)), wp, wb, _stream(stream)))
    return out


# ------------------------------------------------------------------------------------------ time-major [T, N] entry points
def _tm_ws(T, N, like, workspace, stream):
    if workspace is not None:
        return _ws(workspace)
    nbytes = int(lib().rlcs_time_major_workspace_bytes(N, T))
    if not nbytes:
        return None, 0
    # Scratch for this one call; it needs no initialisation.  Freed memory goes back to torch's caching
    # allocator, which reuses it in stream order on the allocating stream; a caller-chosen stream is
    # recorded on the buffer so that the same holds there.
    buf = _torch().empty(nbytes, dtype=_torch().uint8, device=like.device)
    if stream is not None:
        buf.record_stream(stream)
    return buf.data_ptr(), nbytes




def rlcs_gae_time_major(rewards, values, dones, truncs=None, trunc_bootstrap=None, bootstrap=None, *, gamma, lam,
                        advantages=None, returns=None, want_returns=True, workspace=None, stream=None):
    """GAE on [T, N] tensors (element (t, n) at t*N + n); bootstrap [N]."""
    T, N = rewards.shape
    adv = _out(rewards, advantages)
    ret = (_out(rewards, returns) if want_returns else None)
    wp, wb = _tm_ws(T, N, rewards, workspace, stream)
    _check(lib().rlcs_gae_time_major(_ptr(rewards, "f32"), _ptr(values, "f32", (T, N)), _ptr(dones, "u8", (T, N)),
                                     _ptr(truncs, "u8", (T, N)), _ptr(trunc_bootstrap, "f32", (T, N)),
                                     _ptr(bootstrap, "f32", (N,)), _ptr(adv, "f32", (T, N)), _ptr(ret, "f32", (T, N)),
                                     N, T, gamma, lam, wp, wb, _stream(stream)))
    return (adv, ret) if want_returns else adv


def rlcs_vtrace_time_major(rewards, values, log_rhos, dones, truncs=None, trunc_bootstrap=None, bootstrap=None, *,
                           gamma, rho_bar=1.0, c_bar=1.0, vs=None, pg_advantages=None, workspace=None, stream=None):
    T, N = rewards.shape
    vs, adv = _out(rewards, vs), _out(rewards, pg_advantages)
    wp, wb = _tm_ws(T, N, rewards, workspace, stream)
    _check(lib().rlcs_vtrace_time_major(_ptr(rewards, "f32"), _ptr(values, "f32", (T, N)), _ptr(log_rhos, "f32", (T, N)),
                                        _ptr(dones, "u8", (T, N)), _ptr(truncs, "u8", (T, N)),
                                        _ptr(trunc_bootstrap, "f32", (T, N)), _ptr(bootstrap, "f32", (N,)),
                                        _ptr(vs, "f32", (T, N)), _ptr(adv, "f32", (T, N)), N, T, gamma, rho_bar, c_bar,
                                        wp, wb, _stream(stream)))
    return vs, adv


def rlcs_retrace_time_major(rewards, q_sa, expected_q, log_rhos, dones, truncs=None, trunc_bootstrap=None,
                            bootstrap=None, *, gamma, lam, c_bar=1.0, q_targets=None, workspace=None, stream=None):
    T, N = rewards.shape
    out = _out(rewards, q_targets)
    wp, wb = _tm_ws(T, N, rewards, workspace, stream)
    _check(lib().rlcs_retrace_time_major(_ptr(rewards, "f32"), _ptr(q_sa, "f32", (T, N)), _ptr(expected_q, "f32", (T, N)),
                                         _ptr(log_rhos, "f32", (T, N)), _ptr(dones, "u8", (T, N)),
                                         _ptr(truncs, "u8", (T, N)), _ptr(trunc_bootstrap, "f32", (T, N)),
                                         _ptr(bootstrap, "f32", (N,)), _ptr(out, "f32", (T, N)), N, T, gamma, lam, c_bar,
                                         wp, wb, _stream(stream)))
    return out


def rlcs_td_lambda_time_major(rewards, values, dones, truncs=None, trunc_bootstrap=None, bootstrap=None, *, gamma, lam,
                              returns=None, workspace=None, stream=None):
    T, N = rewards.shape
    out = _out(rewards, returns)
    wp, wb = _tm_ws(T, N, rewards, workspace, stream)
    _check(lib().rlcs_td_lambda_time_major(_ptr(rewards, "f32"), _ptr(values, "f32", (T, N)), _ptr(dones, "u8", (T, N)),
                                           _ptr(truncs, "u8", (T, N)), _ptr(trunc_bootstrap, "f32", (T, N)),
                                           _ptr(bootstrap, "f32", (N,)), _ptr(out, "f32", (T, N)), N, T, gamma, lam,
                                           wp, wb, _stream(stream)))
    return out


def rlcs_discounted_return_time_major(rewards, dones, truncs=None, trunc_bootstrap=None, bootstrap=None, *, gamma,
                                      returns=None, workspace=None, stream=None):
    T, N = rewards.shape
    out = _out(rewards, returns)
    wp, wb = _tm_ws(T, N, rewards, workspace, stream)
    _check(lib().rlcs_discounted_return_time_major(_ptr(rewards, "f32"), _ptr(dones, "u8", (T, N)),
                                                   _ptr(truncs, "u8", (T, N)), _ptr(trunc_bootstrap, "f32", (T, N)),
                                                   _ptr(bootstrap, "f32", (N,)), _ptr(out, "f32", (T, N)), N, T, gamma,
                                                   wp, wb, _stream(stream)))
    return out


def rlcs_elig_trace_time_major(x, dones, *, gamma, lam, traces=None, workspace=None, stream=None):
    T, N = x.shape
    out = _out(x, traces)
    wp, wb = _tm_ws(T, N, x, workspace, stream)
    _check(lib().rlcs_elig_trace_time_major(_ptr(x, "f32"), _ptr(dones, "u8", (T, N)), _ptr(out, "f32", (T, N)), N, T,
                                            gamma, lam, wp, wb, _stream(stream)))
    return out


def rlcs_episodic_prefix_sum_time_major(x, dones, *, starts_at=False, sums=None, workspace=None, stream=None):
    T, N = x.shape
    out = _out(x, sums)
    wp, wb = _tm_ws(T, N, x, workspace, stream)
    _check(lib().rlcs_episodic_prefix_sum_time_major(_ptr(x, "f32"), _ptr(dones, "u8", (T, N)), _ptr(out, "f32", (T, N)),
                                                     N, T, int(bool(starts_at)), wp, wb, _stream(stream)))
    return out
