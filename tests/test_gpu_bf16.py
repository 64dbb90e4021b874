"""GPU parity of the bfloat16-tensor entry points (rlcs_*_bf16), called through the C ABI.

Inputs are the seeded rollouts rounded to bfloat16 (so the oracle, in fp64, and the kernels see the
same numbers).  The kernels compute in fp32 and round once on store, hence the bar

    |out - ref| <= tol32 + 2^-8 * (|ref| + tol32),     tol32 = 1e-4 + 1e-5 |ref|

(a correctly rounded bfloat16 of any value within the fp32 tolerance of the exact result: 8
significant bits, half an ulp is at most 2^-8 relative).  A second, sharper check needs no bound:
with the tile shape pinned, the bfloat16 entry point must equal the fp32 entry point's output
rounded to bfloat16 by torch, bit for bit.
"""
import numpy as np
import pytest

from _util import ALL_ALGOS, ATOL, RTOL, guarded_empty, guarded_upload, run_oracle

pytestmark = pytest.mark.gpu

FLOAT_KEYS = ("rewards", "values", "bootstrap", "trunc_bootstrap", "q_sa", "expected_q", "log_rhos", "x")
BACKWARD = ("gae", "vtrace", "retrace", "td_lambda", "discounted_return")
BUILT_VARIANTS = (0, 5, 6, 18, 19, 20, 21)


@pytest.fixture(scope="module")
def W():
    from paper_2608_17641_b200 import workloads
    return workloads


@pytest.fixture(scope="module")
def B():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2608_17641_b200 import binding
    binding.lib()
    binding.rlcs_debug_set_carry_fault(-1, 0)
    binding.rlcs_debug_set_tile_variant(-1)
    return binding


def to_bf16_values(ro):
    """Round every float array of the rollout to the nearest bfloat16 value, in place (fp32 storage)."""
    import torch
    for k in FLOAT_KEYS:
        a = getattr(ro, k)
        if a is not None:
            setattr(ro, k, torch.from_numpy(np.ascontiguousarray(a)).to(torch.bfloat16).to(torch.float32).numpy())
    return ro


class Dev16:
    """Device copies: float arrays as bfloat16 tensors, masks as uint8; `offset` shifts every tensor
    by that many elements from its allocation start (2-byte alignment only when odd)."""

    def __init__(self, ro, offset=0):
        import torch
        self.ro, self.offset = ro, offset

        def up(a, bf16):
            if a is None:
                return None
            return guarded_upload(a, offset, dtype=torch.bfloat16 if bf16 else None)

        for k in FLOAT_KEYS:
            setattr(self, k, up(getattr(ro, k), True))
        self.dones, self.truncs, self.any_done = up(ro.dones, False), up(ro.truncs, False), up(ro.any_done, False)

    def out(self):
        import torch
        return guarded_empty((self.ro.N, self.ro.T), torch.bfloat16, self.offset, label="bf16 output")


def run_gpu16(B, dev, algos=ALL_ALGOS, use_truncs=True, use_bootstrap=True):
    import torch
    ro, p = dev.ro, dev.ro.params
    ws = B.Workspace(ro.N, ro.T)
    tr = dev.truncs if use_truncs else None
    bv = dev.trunc_bootstrap if use_truncs else None
    bt = dev.bootstrap if use_bootstrap else None
    res = {}
    for a in algos:
        if a == "gae":
            res[a] = B.rlcs_gae_bf16(dev.rewards, dev.values, dev.dones, tr, bv, bt, gamma=p["gamma"], lam=p["lam"],
                                     advantages=dev.out(), returns=dev.out(), workspace=ws)
        elif a == "vtrace":
            res[a] = B.rlcs_vtrace_bf16(dev.rewards, dev.values, dev.log_rhos, dev.dones, tr, bv, bt, gamma=p["gamma"],
                                        rho_bar=p["rho_bar"], c_bar=p["c_bar"], vs=dev.out(), pg_advantages=dev.out(),
                                        workspace=ws)
        elif a == "retrace":
            res[a] = B.rlcs_retrace_bf16(dev.rewards, dev.q_sa, dev.expected_q, dev.log_rhos, dev.dones, tr, bv, bt,
                                         gamma=p["gamma"], lam=p["lam"], c_bar=p["c_bar"], q_targets=dev.out(), workspace=ws)
        elif a == "td_lambda":
            res[a] = B.rlcs_td_lambda_bf16(dev.rewards, dev.values, dev.dones, tr, bv, bt, gamma=p["gamma"], lam=p["lam"],
                                           returns=dev.out(), workspace=ws)
        elif a == "discounted_return":
            res[a] = B.rlcs_discounted_return_bf16(dev.rewards, dev.dones, tr, bv, bt, gamma=p["gamma"], returns=dev.out(),
                                                   workspace=ws)
        elif a == "elig_trace":
            res[a] = B.rlcs_elig_trace_bf16(dev.x, dev.any_done, gamma=p["gamma"], lam=p["lam"], traces=dev.out(), workspace=ws)
        elif a == "prefix_ends_at":
            res[a] = B.rlcs_episodic_prefix_sum_bf16(dev.x, dev.any_done, sums=dev.out(), workspace=ws)
        elif a == "prefix_starts_at":
            res[a] = B.rlcs_episodic_prefix_sum_bf16(dev.x, dev.any_done, starts_at=True, sums=dev.out(), workspace=ws)
    torch.cuda.synchronize()
    assert ws.device_status() == 0, "device reported a carry-wait timeout"
    return res


def assert_close16(name, gpu, ref):
    """gpu: bfloat16 tensor; ref: fp64 oracle output."""
    import torch
    assert gpu.dtype == torch.bfloat16 and tuple(gpu.shape) == ref.shape, (name, gpu.dtype, gpu.shape, ref.shape)
    g = gpu.to(torch.float32).cpu().numpy().astype(np.float64)
    assert np.isfinite(g).all(), f"{name}: non-finite output"
    tol32 = ATOL + RTOL * np.abs(ref)
    bound = tol32 + 2.0 ** -8 * (np.abs(ref) + tol32)
    err = np.abs(g - ref)
    bad = err > bound
    if bad.any():
        idx = np.unravel_index(np.argmax(err - bound), err.shape)
        raise AssertionError(f"{name}: {int(bad.sum())} of {bad.size} elements out of tolerance; worst at {idx}: "
                             f"gpu={g[idx]!r} ref={ref[idx]!r} err={err[idx]:.3e} bound={bound[idx]:.3e}")


def compare16(oracle, B, ro, algos=ALL_ALGOS, offset=0, **kw):
    to_bf16_values(ro)
    gpu = run_gpu16(B, Dev16(ro, offset), algos, **kw)
    ref = run_oracle(oracle, ro, algos, **kw)
    for a in algos:
        if isinstance(ref[a], tuple):
            for i, (g, r) in enumerate(zip(gpu[a], ref[a])):
                assert_close16(f"{a}[{i}]", g, r)
        else:
            assert_close16(a, gpu[a], ref[a])
    return gpu


@pytest.mark.parametrize("N,T", [(1, 1), (3, 7), (5, 1001), (64, 512), (256, 128), (7, 5000), (2, 40000), (4096, 64)])
@pytest.mark.parametrize("p_flag", [0.0, 0.02, 0.3])
def test_bf16_shape_matrix(oracle, W, B, N, T, p_flag):
    compare16(oracle, B, W.make_rollout(120, N, T, p_done=p_flag, p_trunc=p_flag / 2, salt=N * 7919 + T))


def test_bf16_null_bootstrap_and_null_truncs(oracle, W, B):
    ro = W.make_rollout(121, 6, 900, p_done=0.02, p_trunc=0.02)
    compare16(oracle, B, ro, algos=BACKWARD, use_bootstrap=False)
    compare16(oracle, B, ro, algos=BACKWARD, use_truncs=False)


@pytest.mark.parametrize("offset", [1, 3, 8])
def test_bf16_unaligned_pointers_take_elementwise_path(oracle, W, B, offset):
    compare16(oracle, B, W.make_rollout(122, 9, 777, salt=offset), offset=offset)


@pytest.mark.parametrize("N,T", [(4, 2048), (3, 8192), (2, 16384)])
def test_bf16_rows_of_whole_tiles_use_the_cluster_carry(oracle, W, B, N, T):
    compare16(oracle, B, W.make_rollout(123, N, T, p_done=0.001, p_trunc=0.001), algos=("gae", "discounted_return", "elig_trace"))


@pytest.mark.parametrize("N,T", [(6, 6016), (3, 16384), (40, 2000), (9, 1000)])
def test_bf16_row_kernels(oracle, W, B, N, T):
    """The layouts without a carry between blocks on bfloat16 tensors: one thread block per row (forced
    here, few rows) and row-aligned tiles."""
    B.rlcs_debug_set_row_blocks(1)
    try:
        compare16(oracle, B, W.make_rollout(127, N, T, p_done=0.002, p_trunc=0.002))
    finally:
        B.rlcs_debug_set_row_blocks(-1)


def test_bf16_large_problem_with_carry(oracle, W, B):
    """Above 2^23 steps the 16-steps-per-thread tile is chosen; T = 3000 makes rows straddle tiles."""
    compare16(oracle, B, W.make_rollout(124, 2900, 3000, p_done=0.002, p_trunc=0.002), algos=("gae", "vtrace", "retrace"))


def test_bf16_full_size_sampled_rows(oracle, W, B):
    """16384 x 2048 with truncations, the configuration bench.py times: GAE, V-Trace and the discounted
    return on bfloat16 tensors; every element of 192 sampled rows against the oracle."""
    import copy
    import torch
    ro = to_bf16_values(W.config5())
    p = ro.params
    rows = np.unique(np.concatenate([[0, ro.N - 1], np.random.default_rng(7).integers(0, ro.N, 190)]))
    small = copy.copy(ro)
    for k in FLOAT_KEYS + ("dones", "truncs"):
        a = getattr(ro, k)
        setattr(small, k, None if a is None else np.ascontiguousarray(a[rows]))
    small.N = len(rows)
    ref = run_oracle(oracle, small, ("gae", "vtrace", "discounted_return"))
    dev = Dev16(ro)
    ws = B.Workspace(ro.N, ro.T)
    idx = guarded_upload(rows)
    adv, ret = B.rlcs_gae_bf16(dev.rewards, dev.values, dev.dones, dev.truncs, dev.trunc_bootstrap, dev.bootstrap,
                               gamma=p["gamma"], lam=p["lam"], workspace=ws)
    assert_close16("gae", adv[idx], ref["gae"][0]); assert_close16("ret", ret[idx], ref["gae"][1])
    vs, pg = B.rlcs_vtrace_bf16(dev.rewards, dev.values, dev.log_rhos, dev.dones, dev.truncs, dev.trunc_bootstrap,
                                dev.bootstrap, gamma=p["gamma"], rho_bar=p["rho_bar"], c_bar=p["c_bar"], workspace=ws)
    assert_close16("vs", vs[idx], ref["vtrace"][0]); assert_close16("pg", pg[idx], ref["vtrace"][1])
    out = B.rlcs_discounted_return_bf16(dev.rewards, dev.dones, dev.truncs, dev.trunc_bootstrap, dev.bootstrap,
                                        gamma=p["gamma"], workspace=ws)
    assert_close16("disc", out[idx], ref["discounted_return"])
    torch.cuda.synchronize()
    assert ws.device_status() == 0


@pytest.mark.parametrize("variant", BUILT_VARIANTS)
def test_bf16_equals_rounded_fp32_bit_for_bit(oracle, W, B, variant):
    """Same tile shape, same fp32 arithmetic: the only difference is the rounding on store, and torch's
    float32 -> bfloat16 conversion (round to nearest even) must reproduce it exactly."""
    import torch
    ro = to_bf16_values(W.make_rollout(125, 37, 2500, p_done=0.01, p_trunc=0.01, salt=variant))
    p = ro.params
    d16 = Dev16(ro)
    f32 = lambda t: None if t is None else t.to(torch.float32)
    ws = B.Workspace(ro.N, ro.T)
    B.rlcs_debug_set_tile_variant(variant)
    try:
        a16, r16 = B.rlcs_gae_bf16(d16.rewards, d16.values, d16.dones, d16.truncs, d16.trunc_bootstrap, d16.bootstrap,
                                   gamma=p["gamma"], lam=p["lam"], workspace=ws)
        a32, r32 = B.rlcs_gae(f32(d16.rewards), f32(d16.values), d16.dones, d16.truncs, f32(d16.trunc_bootstrap),
                              f32(d16.bootstrap), gamma=p["gamma"], lam=p["lam"], workspace=ws)
        q16 = B.rlcs_retrace_bf16(d16.rewards, d16.q_sa, d16.expected_q, d16.log_rhos, d16.dones, d16.truncs,
                                  d16.trunc_bootstrap, d16.bootstrap, gamma=p["gamma"], lam=p["lam"], workspace=ws)
        q32 = B.rlcs_retrace(f32(d16.rewards), f32(d16.q_sa), f32(d16.expected_q), f32(d16.log_rhos), d16.dones, d16.truncs,
                             f32(d16.trunc_bootstrap), f32(d16.bootstrap), gamma=p["gamma"], lam=p["lam"], workspace=ws)
        z16 = B.rlcs_elig_trace_bf16(d16.x, d16.any_done, gamma=p["gamma"], lam=p["lam"], workspace=ws)
        z32 = B.rlcs_elig_trace(f32(d16.x), d16.any_done, gamma=p["gamma"], lam=p["lam"], workspace=ws)
    finally:
        B.rlcs_debug_set_tile_variant(-1)
    for name, g, r in (("adv", a16, a32), ("ret", r16, r32), ("retrace", q16, q32), ("elig", z16, z32)):
        assert torch.equal(g.view(torch.int16), r.to(torch.bfloat16).view(torch.int16)), name


def test_bf16_randomized_shapes_flags_variants_and_options(oracle, W, B):
    rng = np.random.default_rng(20260819)
    for case in range(40):
        N = int(rng.integers(1, 200))
        T = int(rng.choice([rng.integers(1, 40), rng.integers(40, 3000), rng.integers(3000, 12000)]))
        if N * T > 600_000:
            N = max(1, 600_000 // T)
        ro = W.make_rollout(126, N, T, p_done=float(rng.choice([0.0, 0.001, 0.02, 0.3])),
                            p_trunc=float(rng.choice([0.0, 0.005, 0.2])), salt=case)
        ro.params.update(gamma=float(rng.choice([0.9, 0.99, 1.0])), lam=float(rng.choice([0.0, 0.5, 0.95, 1.0])),
                         rho_bar=float(rng.choice([0.5, 1.0, 2.0])), c_bar=float(rng.choice([0.5, 1.0])))
        variant = int(rng.choice((-1,) + BUILT_VARIANTS))
        B.rlcs_debug_set_tile_variant(variant)
        try:
            compare16(oracle, B, ro, offset=int(rng.choice([0, 0, 0, 1, 3, 16])),
                      use_truncs=bool(rng.random() < 0.7), use_bootstrap=bool(rng.random() < 0.8))
        except AssertionError as e:
            raise AssertionError(f"case {case}: N={N} T={T} variant={variant}: {e}")
        finally:
            B.rlcs_debug_set_tile_variant(-1)


def test_bf16_argument_checks(B):
    L = B.lib()
    P = 0x7f0000000000
    g = lambda **k: L.rlcs_gae_bf16(k.get("r", P), P, k.get("d", P), k.get("tr"), k.get("bv"), None, P, None,
                                    k.get("N", 4), k.get("T", 128), k.get("g", 0.9), 0.9, None, 0, None)
    assert g(N=0) == B.RLCS_OK and g(N=-1) == B.RLCS_ERR_SIZE and g(g=2.0) == B.RLCS_ERR_ARG
    assert g(r=None) == B.RLCS_ERR_NULL and g(d=None) == B.RLCS_ERR_NULL and g(tr=P) == B.RLCS_ERR_NULL
    assert g(r=P + 1) == B.RLCS_ERR_ALIGN                 # bfloat16 tensors need 2-byte alignment
    assert g(N=3, T=3000) == B.RLCS_ERR_WORKSPACE         # rows straddle tiles: the carry needs a workspace
