"""Sequential fp64 CPU oracle (test infrastructure, not part of the product).

Thin numpy/ctypes front end of ``rlcs_oracle.c``: every routine walks one row
at a time, one timestep at a time, in double precision.  Only ``tests/``, the
smoke check and the benchmark's CPU legs may import this package; the CUDA
library never does, and this package never imports the CUDA library.

Scalar parameters (gamma, lambda, clips) are rounded to fp32 first, because
the library's C signatures fix them as ``float``; the oracle then computes with
that value widened to fp64.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading
from concurrent.futures import ThreadPoolExecutor

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "rlcs_oracle.c")
_LIB = os.path.join(_HERE, "librlcs_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain -O2, no fast-math, no contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-ffp-contract=off", "-Wall", "-Wextra",
             "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_F = ctypes.POINTER(ctypes.c_float)
_U = ctypes.POINTER(ctypes.c_uint8)
_D = ctypes.POINTER(ctypes.c_double)
_i64 = ctypes.c_int64
_dbl = ctypes.c_double


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            lib.rlcs_oracle_gae.argtypes = [_F, _F, _U, _U, _F, _F, _D, _D, _i64, _i64, _dbl, _dbl]
            lib.rlcs_oracle_td_lambda.argtypes = [_F, _F, _U, _U, _F, _F, _D, _i64, _i64, _dbl, _dbl]
            lib.rlcs_oracle_discounted_return.argtypes = [_F, _U, _U, _F, _F, _D, _i64, _i64, _dbl]
            lib.rlcs_oracle_vtrace.argtypes = [_F, _F, _F, _U, _U, _F, _F, _D, _D, _i64, _i64, _dbl, _dbl, _dbl]
            lib.rlcs_oracle_retrace.argtypes = [_F, _F, _F, _F, _U, _U, _F, _F, _D, _i64, _i64, _dbl, _dbl, _dbl]
            lib.rlcs_oracle_retrace_probs.argtypes = [_F, _F, _F, _F, ctypes.POINTER(ctypes.c_int32), _U, _U, _F, _F, _D,
                                                      _i64, _i64, _i64, _dbl, _dbl, _dbl]
            lib.rlcs_oracle_retrace_probs.restype = None
            lib.rlcs_oracle_elig_trace.argtypes = [_F, _U, _D, _i64, _i64, _dbl, _dbl]
            lib.rlcs_oracle_gae_skip.argtypes = [_F, _F, _U, _U, _F, _F, _U, _D, _D, _D, _i64, _i64, _dbl, _dbl]
            lib.rlcs_oracle_gae_skip.restype = None
            lib.rlcs_oracle_elig_trace_vec.argtypes = [_F, _U, _D, _i64, _i64, _i64, _dbl, _dbl]
            lib.rlcs_oracle_elig_trace_vec.restype = None
            lib.rlcs_oracle_elig_trace_vec_beta.argtypes = [_F, _F, _U, _D, _i64, _i64, _i64]
            lib.rlcs_oracle_elig_trace_vec_beta.restype = None
            lib.rlcs_oracle_episodic_prefix_sum.argtypes = [_F, _U, _D, _i64, _i64, ctypes.c_int]
            lib.rlcs_oracle_linear_recurrence.argtypes = [_D, _D, _dbl, _D, _i64, ctypes.c_int]
            lib.rlcs_oracle_combine.argtypes = [_dbl, _dbl, _dbl, _dbl, _D, _D]
            for name in ("gae", "td_lambda", "discounted_return", "vtrace", "retrace", "elig_trace",
                         "episodic_prefix_sum", "linear_recurrence", "combine"):
                getattr(lib, "rlcs_oracle_" + name).restype = None
            _lib = lib
    return _lib


def _f32(a, shape=None):
    if a is None:
        return None
    a = np.ascontiguousarray(a, dtype=np.float32)
    if shape is not None and a.shape != shape:
        raise ValueError(f"expected shape {shape}, got {a.shape}")
    return a


def _u8(a, shape=None):
    if a is None:
        return None
    a = np.asarray(a)
    if a.dtype == np.bool_:
        a = a.astype(np.uint8)
    a = np.ascontiguousarray(a, dtype=np.uint8)
    if shape is not None and a.shape != shape:
        raise ValueError(f"expected shape {shape}, got {a.shape}")
    return a


def _p(a, ty):
    return None if a is None else a.ctypes.data_as(ty)


def _s(x) -> float:
    """fp32-round a scalar parameter (the library's signatures take float)."""
    return float(np.float32(x))


def _shape2(a):
    a = np.asarray(a)
    if a.ndim != 2:
        raise ValueError("expected a [num_envs, T] array")
    return a.shape


def _trunc_args(truncs, trunc_bootstrap, shape):
    if (truncs is None) != (trunc_bootstrap is None):
        raise ValueError("truncs and trunc_bootstrap must be given together")
    return _u8(truncs, shape), _f32(trunc_bootstrap, shape)


def gae(rewards, values, dones, truncs=None, trunc_bootstrap=None, bootstrap=None, *, gamma, lam,
        want_returns=True):
    """GAE advantages (and returns = A + V) -- Section 3.3.1 with the boundary rules of Section 3.2."""
    shape = _shape2(rewards)
    N, T = shape
    r, v, d = _f32(rewards, shape), _f32(values, shape), _u8(dones, shape)
    tr, bv = _trunc_args(truncs, trunc_bootstrap, shape)
    bt = _f32(bootstrap, (N,))
    adv = np.empty(shape, np.float64)
    ret = np.empty(shape, np.float64) if want_returns else None
    _load().rlcs_oracle_gae(_p(r, _F), _p(v, _F), _p(d, _U), _p(tr, _U), _p(bv, _F), _p(bt, _F),
                            _p(adv, _D), _p(ret, _D), N, T, _s(gamma), _s(lam))
    return (adv, ret) if want_returns else adv


def gae_skip(rewards, values, dones, truncs=None, trunc_bootstrap=None, bootstrap=None, *, skip, gamma, lam):
    """GAE with observation-skip masking (Section 9.2, planned): masked steps (skip != 0) are
    transparent.  Returns (advantages, returns = A + W, filled values W)."""
    shape = _shape2(rewards)
    N, T = shape
    r, v, d = _f32(rewards, shape), _f32(values, shape), _u8(dones, shape)
    tr, bv = _trunc_args(truncs, trunc_bootstrap, shape)
    bt = _f32(bootstrap, (N,))
    sk = _u8(skip, shape)
    adv, ret, fil = (np.empty(shape, np.float64) for _ in range(3))
    _load().rlcs_oracle_gae_skip(_p(r, _F), _p(v, _F), _p(d, _U), _p(tr, _U), _p(bv, _F), _p(bt, _F), _p(sk, _U),
                                 _p(adv, _D), _p(ret, _D), _p(fil, _D), N, T, _s(gamma), _s(lam))
    return adv, ret, fil


def gae_normalized(rewards, values, dones, truncs=None, trunc_bootstrap=None, bootstrap=None, *, gamma, lam,
                   eps=1e-8, ddof=1):
    """GAE, then (A - mean) / (std + eps) over all N*T steps; std with `ddof` (0 when N*T <= ddof).
    The paper only names this step (planned extension, Section 9.3); this is the usual PPO convention.
    Plain fp64 sums; returns (normalised advantages, returns = A + V from the raw A)."""
    adv, ret = gae(rewards, values, dones, truncs, trunc_bootstrap, bootstrap, gamma=gamma, lam=lam)
    n = adv.size
    mean = adv.sum() / n
    dev2 = ((adv - mean) ** 2).sum()
    std = np.sqrt(dev2 / (n - ddof)) if n > ddof else 0.0
    return (adv - mean) / (std + float(np.float32(eps))), ret


def td_lambda(rewards, values, dones, truncs=None, trunc_bootstrap=None, bootstrap=None, *, gamma, lam):
    """TD(lambda) returns -- Section 3.3.4."""
    shape = _shape2(rewards)
    N, T = shape
    r, v, d = _f32(rewards, shape), _f32(values, shape), _u8(dones, shape)
    tr, bv = _trunc_args(truncs, trunc_bootstrap, shape)
    bt = _f32(bootstrap, (N,))
    out = np.empty(shape, np.float64)
    _load().rlcs_oracle_td_lambda(_p(r, _F), _p(v, _F), _p(d, _U), _p(tr, _U), _p(bv, _F), _p(bt, _F),
                                  _p(out, _D), N, T, _s(gamma), _s(lam))
    return out


def discounted_return(rewards, dones, truncs=None, trunc_bootstrap=None, bootstrap=None, *, gamma):
    """Discounted returns -- Section 3.3.4 (lambda = 1, no value function)."""
    shape = _shape2(rewards)
    N, T = shape
    r, d = _f32(rewards, shape), _u8(dones, shape)
    tr, bv = _trunc_args(truncs, trunc_bootstrap, shape)
    bt = _f32(bootstrap, (N,))
    out = np.empty(shape, np.float64)
    _load().rlcs_oracle_discounted_return(_p(r, _F), _p(d, _U), _p(tr, _U), _p(bv, _F), _p(bt, _F),
                                          _p(out, _D), N, T, _s(gamma))
    return out


def vtrace(rewards, values, log_rhos, dones, truncs=None, trunc_bootstrap=None, bootstrap=None, *,
           gamma, rho_bar=1.0, c_bar=1.0):
    """V-Trace targets vs and policy-gradient advantages -- Section 3.3.2."""
    shape = _shape2(rewards)
    N, T = shape
    r, v, lr, d = _f32(rewards, shape), _f32(values, shape), _f32(log_rhos, shape), _u8(dones, shape)
    tr, bv = _trunc_args(truncs, trunc_bootstrap, shape)
    bt = _f32(bootstrap, (N,))
    vs = np.empty(shape, np.float64)
    adv = np.empty(shape, np.float64)
    _load().rlcs_oracle_vtrace(_p(r, _F), _p(v, _F), _p(lr, _F), _p(d, _U), _p(tr, _U), _p(bv, _F),
                               _p(bt, _F), _p(vs, _D), _p(adv, _D), N, T, _s(gamma), _s(rho_bar),
                               _s(c_bar))
    return vs, adv


def retrace(rewards, q_sa, expected_q, log_rhos, dones, truncs=None, trunc_bootstrap=None,
            bootstrap=None, *, gamma, lam, c_bar=1.0):
    """Retrace(lambda) Q targets -- Section 3.3.3."""
    shape = _shape2(rewards)
    N, T = shape
    r, q, eq = _f32(rewards, shape), _f32(q_sa, shape), _f32(expected_q, shape)
    lr, d = _f32(log_rhos, shape), _u8(dones, shape)
    tr, bv = _trunc_args(truncs, trunc_bootstrap, shape)
    bt = _f32(bootstrap, (N,))
    out = np.empty(shape, np.float64)
    _load().rlcs_oracle_retrace(_p(r, _F), _p(q, _F), _p(eq, _F), _p(lr, _F), _p(d, _U), _p(tr, _U),
                                _p(bv, _F), _p(bt, _F), _p(out, _D), N, T, _s(gamma), _s(lam),
                                _s(c_bar))
    return out


def retrace_probs(rewards, q_values, target_probs, behaviour_probs, actions, dones, truncs=None,
                  trunc_bootstrap=None, bootstrap=None, *, gamma, lam, c_bar=1.0):
    """Retrace(lambda) Q targets from [N,T,A] Q-values / policy probabilities and actions [N,T]."""
    shape = _shape2(rewards)
    N, T = shape
    A = np.asarray(q_values).shape[2]
    r, d = _f32(rewards, shape), _u8(dones, shape)
    q, pi, mu = _f32(q_values, (N, T, A)), _f32(target_probs, (N, T, A)), _f32(behaviour_probs, (N, T, A))
    act = np.ascontiguousarray(actions, dtype=np.int32)
    if act.shape != shape or act.min() < 0 or act.max() >= A:
        raise ValueError("actions must be [N, T] with values in [0, A)")
    tr, bv = _trunc_args(truncs, trunc_bootstrap, shape)
    bt = _f32(bootstrap, (N,))
    out = np.empty(shape, np.float64)
    _load().rlcs_oracle_retrace_probs(_p(r, _F), _p(q, _F), _p(pi, _F), _p(mu, _F),
                                      act.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)), _p(d, _U), _p(tr, _U),
                                      _p(bv, _F), _p(bt, _F), _p(out, _D), N, T, A, _s(gamma), _s(lam), _s(c_bar))
    return out


def elig_trace(x, dones, *, gamma, lam):
    """Scalar eligibility trace, forward -- Section 3.3.5."""
    shape = _shape2(x)
    N, T = shape
    xx, d = _f32(x, shape), _u8(dones, shape)
    out = np.empty(shape, np.float64)
    _load().rlcs_oracle_elig_trace(_p(xx, _F), _p(d, _U), _p(out, _D), N, T, _s(gamma), _s(lam))
    return out


def elig_trace_vec(x, dones, *, gamma, lam):
    """Vector-valued eligibility trace: x [N,T,D], dones [N,T] -- Table 1 (vector form), Section 3.3.5."""
    xx = np.ascontiguousarray(x, dtype=np.float32)
    if xx.ndim != 3:
        raise ValueError("expected an [N, T, D] array")
    N, T, D = xx.shape
    d = _u8(dones, (N, T))
    out = np.empty(xx.shape, np.float64)
    _load().rlcs_oracle_elig_trace_vec(_p(xx, _F), _p(d, _U), _p(out, _D), N, T, D, _s(gamma), _s(lam))
    return out


def elig_trace_vec_beta(x, beta, dones):
    """Eligibility trace with a decay per component and step: x, beta [N,T,D], dones [N,T] -- Eq. 1
    component by component (per-dimension beta, Section 9.1)."""
    xx = np.ascontiguousarray(x, dtype=np.float32)
    if xx.ndim != 3:
        raise ValueError("expected an [N, T, D] array")
    N, T, D = xx.shape
    bb = np.ascontiguousarray(beta, dtype=np.float32)
    if bb.shape != xx.shape:
        raise ValueError("beta must have the shape of x")
    d = _u8(dones, (N, T))
    out = np.empty(xx.shape, np.float64)
    _load().rlcs_oracle_elig_trace_vec_beta(_p(xx, _F), _p(bb, _F), _p(d, _U), _p(out, _D), N, T, D)
    return out


def episodic_prefix_sum(x, dones, *, starts_at=False):
    """Episodic prefix sum, forward -- Section 3.3.6 (both boundary conventions)."""
    shape = _shape2(x)
    N, T = shape
    xx, d = _f32(x, shape), _u8(dones, shape)
    out = np.empty(shape, np.float64)
    _load().rlcs_oracle_episodic_prefix_sum(_p(xx, _F), _p(d, _U), _p(out, _D), N, T, int(bool(starts_at)))
    return out


def linear_recurrence(alpha, beta, carry=0.0, *, forward=False):
    """Eq. 1 on one row of fp64 coefficients (backward, or the forward mirror)."""
    a = np.ascontiguousarray(alpha, dtype=np.float64)
    b = np.ascontiguousarray(beta, dtype=np.float64)
    if a.ndim != 1 or a.shape != b.shape:
        raise ValueError("alpha and beta must be 1-D and of equal length")
    out = np.empty_like(a)
    _load().rlcs_oracle_linear_recurrence(_p(a, _D), _p(b, _D), float(carry), _p(out, _D), a.shape[0],
                                          int(bool(forward)))
    return out


def combine(B, A):
    """Eq. 2: B (+) A with B = (alpha_B, beta_B) the chronologically earlier pair."""
    oa, ob = ctypes.c_double(), ctypes.c_double()
    _load().rlcs_oracle_combine(float(B[0]), float(B[1]), float(A[0]), float(A[1]),
                                ctypes.byref(oa), ctypes.byref(ob))
    return oa.value, ob.value


def run_rows_parallel(fn, arrays_2d: dict, arrays_1d: dict, threads: int, **params):
    """Run ``fn`` on contiguous row blocks in ``threads`` host threads (rows are independent).

    ``arrays_2d`` / ``arrays_1d`` map keyword names to [N,T] / [N] arrays (or None); outputs of the
    blocks are concatenated along rows.  ctypes releases the GIL during each C call.
    """
    N = next(a for a in arrays_2d.values() if a is not None).shape[0]
    threads = max(1, min(threads, N))
    bounds = np.linspace(0, N, threads + 1).astype(np.int64)

    def work(k):
        lo, hi = int(bounds[k]), int(bounds[k + 1])
        kw = {k2: (None if a is None else a[lo:hi]) for k2, a in arrays_2d.items()}
        kw.update({k1: (None if a is None else a[lo:hi]) for k1, a in arrays_1d.items()})
        return fn(**kw, **params)

    if threads == 1:
        return work(0)
    with ThreadPoolExecutor(threads) as ex:
        parts = list(ex.map(work, range(threads)))
    if isinstance(parts[0], tuple):
        return tuple(np.concatenate([p[i] for p in parts], axis=0) for i in range(len(parts[0])))
    return np.concatenate(parts, axis=0)
