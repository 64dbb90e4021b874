"""Shared helpers of the GPU parity tests: upload a Rollout, run all algorithms on the GPU through
the C ABI binding and on the CPU oracle, and compare element by element."""
from __future__ import annotations

import numpy as np

ATOL, RTOL = 1e-4, 1e-5          # the stated bar: |gpu - ref| <= 1e-4 + 1e-5 |ref|

ALL_ALGOS = ("gae", "vtrace", "retrace", "td_lambda", "discounted_return", "elig_trace",
             "prefix_ends_at", "prefix_starts_at")


def assert_close(name, gpu, ref):
    """gpu: fp32 array (numpy); ref: fp64 oracle output."""
    gpu = np.asarray(gpu)
    assert gpu.dtype == np.float32 and gpu.shape == ref.shape, (name, gpu.dtype, gpu.shape, ref.shape)
    assert np.isfinite(gpu).all(), f"{name}: non-finite output"
    err = np.abs(gpu.astype(np.float64) - ref)
    bound = ATOL + RTOL * np.abs(ref)
    bad = err > bound
    if bad.any():
        idx = np.unravel_index(np.argmax(err - bound), err.shape)
        raise AssertionError(f"{name}: {int(bad.sum())} of {bad.size} elements out of tolerance; worst at {idx}: "
                             f"gpu={gpu[idx]!r} ref={ref[idx]!r} err={err[idx]:.3e}")
    return float(err.max())


# ---------------------------------------------------------------------------------------------- guard bands
# Every device tensor the tests hand to the library sits between two bands of 0xFF bytes (a NaN
# pattern for fp32 and bfloat16, 255 for masks, -1 for int32).  A kernel that writes outside a
# tensor -- before it, behind it, or into an input -- lands in a band; the bands of all live
# allocations are compared after every run_gpu() and at the end of every GPU test (conftest.py).
GUARD = 64                       # elements on each side
_live = []                       # (flat uint8 view, first payload byte, one-past-last payload byte, label)


def guarded_empty(shape, dtype, offset: int = 0, label: str = ""):
    """Uninitialised device tensor of `shape` inside guard bands; `offset` shifts it by that many
    elements from the (512-byte aligned) allocation start + GUARD elements, to break alignment."""
    import torch
    n = 1
    for d in (shape if isinstance(shape, (tuple, list, torch.Size)) else (shape,)):
        n *= int(d)
    flat = torch.empty(GUARD + offset + n + GUARD, dtype=dtype, device="cuda")
    raw = flat.view(torch.uint8)
    raw.fill_(0xFF)
    es = flat.element_size()
    _live.append((raw, (GUARD + offset) * es, (GUARD + offset + n) * es, label or str(tuple(shape) if hasattr(shape, "__len__") else shape)))
    return flat[GUARD + offset:GUARD + offset + n].view(shape)


def guarded_upload(a, offset: int = 0, dtype=None, label: str = ""):
    """Device copy of a numpy array (or CPU tensor) inside guard bands; None stays None."""
    import torch
    if a is None:
        return None
    t = a if isinstance(a, torch.Tensor) else torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    out = guarded_empty(tuple(t.shape), t.dtype, offset, label)
    out.copy_(t)
    return out


def check_guards(clear: bool = False):
    """Assert that no guard band of a live allocation has been written."""
    import torch
    if _live and torch.cuda.is_available():
        torch.cuda.synchronize()
        for raw, lo, hi, label in _live:
            ok = bool(raw[:lo].eq(0xFF).all().item()) and bool(raw[hi:].eq(0xFF).all().item())
            if not ok:
                front = int((raw[:lo] != 0xFF).sum().item())
                back = int((raw[hi:] != 0xFF).sum().item())
                if clear:
                    _live.clear()
                raise AssertionError(f"guard band overwritten around tensor {label}: {front} bytes before it, {back} bytes behind it")
    if clear:
        _live.clear()


class Dev:
    """Device copies of a Rollout's arrays (torch tensors), each inside guard bands; `offset` shifts
    every tensor by that many elements from its aligned position to break 16-byte alignment."""

    def __init__(self, ro, offset: int = 0):
        self.ro = ro
        self.offset = offset
        for k in ("rewards", "values", "dones", "bootstrap", "truncs", "trunc_bootstrap", "q_sa", "expected_q",
                  "log_rhos", "x"):
            setattr(self, k, guarded_upload(getattr(ro, k), offset, label=k))
        self.any_done = guarded_upload(ro.any_done, offset, label="any_done")

    def empty_out(self):
        import torch
        return guarded_empty((self.ro.N, self.ro.T), torch.float32, self.offset, label="output")


def run_gpu(dev: Dev, algos=ALL_ALGOS, workspace="auto", use_truncs=True, use_bootstrap=True):
    """Run the chosen algorithms through the binding; returns {name: numpy fp32 array or tuple}."""
    from paper_2608_17641_b200 import binding as B
    ro = dev.ro
    p = ro.params
    ws = B.Workspace(ro.N, ro.T) if workspace == "auto" else workspace
    tr = dev.truncs if use_truncs else None
    bv = dev.trunc_bootstrap if use_truncs else None
    bt = dev.bootstrap if use_bootstrap else None
    o = lambda: dict(workspace=ws)
    res = {}
    for a in algos:
        if a == "gae":
            adv, ret = B.rlcs_gae(dev.rewards, dev.values, dev.dones, tr, bv, bt, gamma=p["gamma"], lam=p["lam"],
                                  advantages=dev.empty_out(), returns=dev.empty_out(), **o())
            res[a] = (adv, ret)
        elif a == "vtrace":
            res[a] = B.rlcs_vtrace(dev.rewards, dev.values, dev.log_rhos, dev.dones, tr, bv, bt, gamma=p["gamma"],
                                   rho_bar=p["rho_bar"], c_bar=p["c_bar"], vs=dev.empty_out(),
                                   pg_advantages=dev.empty_out(), **o())
        elif a == "retrace":
            res[a] = B.rlcs_retrace(dev.rewards, dev.q_sa, dev.expected_q, dev.log_rhos, dev.dones, tr, bv, bt,
                                    gamma=p["gamma"], lam=p["lam"], c_bar=p["c_bar"], q_targets=dev.empty_out(), **o())
        elif a == "td_lambda":
            res[a] = B.rlcs_td_lambda(dev.rewards, dev.values, dev.dones, tr, bv, bt, gamma=p["gamma"], lam=p["lam"],
                                      returns=dev.empty_out(), **o())
        elif a == "discounted_return":
            res[a] = B.rlcs_discounted_return(dev.rewards, dev.dones, tr, bv, bt, gamma=p["gamma"],
                                              returns=dev.empty_out(), **o())
        elif a == "elig_trace":
            res[a] = B.rlcs_elig_trace(dev.x, dev.any_done, gamma=p["gamma"], lam=p["lam"], traces=dev.empty_out(), **o())
        elif a == "prefix_ends_at":
            res[a] = B.rlcs_episodic_prefix_sum(dev.x, dev.any_done, sums=dev.empty_out(), **o())
        elif a == "prefix_starts_at":
            res[a] = B.rlcs_episodic_prefix_sum(dev.x, dev.any_done, starts_at=True, sums=dev.empty_out(), **o())
        else:
            raise KeyError(a)
    import torch
    torch.cuda.synchronize()
    check_guards()
    if ws is not None:
        assert ws.device_status() == 0, "device reported a carry-wait timeout"
    to_np = lambda v: tuple(t.cpu().numpy() for t in v) if isinstance(v, tuple) else v.cpu().numpy()
    return {k: to_np(v) for k, v in res.items()}


def run_oracle(oracle, ro, algos=ALL_ALGOS, use_truncs=True, use_bootstrap=True, threads=8):
    p = ro.params
    tr = ro.truncs if use_truncs else None
    bv = ro.trunc_bootstrap if use_truncs else None
    bt = ro.bootstrap if use_bootstrap else None
    d_fwd = ro.any_done
    bw2 = dict(dones=ro.dones, truncs=tr, trunc_bootstrap=bv)
    bw1 = dict(bootstrap=bt)
    par = lambda fn, a2, a1, **kw: oracle.run_rows_parallel(fn, a2, a1, threads, **kw)
    res = {}
    for a in algos:
        if a == "gae":
            res[a] = par(oracle.gae, dict(rewards=ro.rewards, values=ro.values, **bw2), bw1, gamma=p["gamma"], lam=p["lam"])
        elif a == "vtrace":
            res[a] = par(oracle.vtrace, dict(rewards=ro.rewards, values=ro.values, log_rhos=ro.log_rhos, **bw2), bw1,
                         gamma=p["gamma"], rho_bar=p["rho_bar"], c_bar=p["c_bar"])
        elif a == "retrace":
            res[a] = par(oracle.retrace, dict(rewards=ro.rewards, q_sa=ro.q_sa, expected_q=ro.expected_q,
                                              log_rhos=ro.log_rhos, **bw2), bw1, gamma=p["gamma"], lam=p["lam"],
                         c_bar=p["c_bar"])
        elif a == "td_lambda":
            res[a] = par(oracle.td_lambda, dict(rewards=ro.rewards, values=ro.values, **bw2), bw1, gamma=p["gamma"], lam=p["lam"])
        elif a == "discounted_return":
            res[a] = par(oracle.discounted_return, dict(rewards=ro.rewards, **bw2), bw1, gamma=p["gamma"])
        elif a == "elig_trace":
            res[a] = par(oracle.elig_trace, dict(x=ro.x, dones=d_fwd), {}, gamma=p["gamma"], lam=p["lam"])
        elif a == "prefix_ends_at":
            res[a] = par(oracle.episodic_prefix_sum, dict(x=ro.x, dones=d_fwd), {})
        elif a == "prefix_starts_at":
            res[a] = par(oracle.episodic_prefix_sum, dict(x=ro.x, dones=d_fwd), {}, starts_at=True)
    return res


def compare_all(oracle, ro, algos=ALL_ALGOS, offset=0, **kw):
    dev = Dev(ro, offset=offset)
    gpu = run_gpu(dev, algos, **kw)
    okw = {k: v for k, v in kw.items() if k in ("use_truncs", "use_bootstrap")}
    ref = run_oracle(oracle, ro, algos, **okw)
    worst = {}
    for a in algos:
        if isinstance(ref[a], tuple):
            worst[a] = max(assert_close(f"{a}[{i}]", g, r) for i, (g, r) in enumerate(zip(gpu[a], ref[a])))
        else:
            worst[a] = assert_close(a, gpu[a], ref[a])
    return gpu, ref, worst
