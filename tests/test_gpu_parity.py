"""GPU parity: the CUDA path, called through the C ABI, against the fp64 CPU oracle on the same
seeded inputs.  Bar: |gpu - ref| <= 1e-4 + 1e-5 |ref| element by element; segmentation exact."""
import os

import numpy as np
import pytest

from _util import (ALL_ALGOS, Dev, assert_close, check_guards, compare_all, guarded_empty, guarded_upload, run_gpu,
                   run_oracle)

pytestmark = pytest.mark.gpu

# The suite runs on the library's default kernel; RLCS_TEST_VARIANT=<n> reruns all of it on variant n.
BASE_VARIANT = int(os.environ.get("RLCS_TEST_VARIANT", "-1"))

BACKWARD = ("gae", "vtrace", "retrace", "td_lambda", "discounted_return")


@pytest.fixture(scope="module")
def W():
    from paper_2608_17641_b200 import workloads
    return workloads


@pytest.fixture(scope="module")
def B():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2608_17641_b200 import binding
    binding.lib()                      # fail loudly if the extension is missing
    binding.rlcs_debug_set_carry_fault(-1, 0)
    binding.rlcs_debug_set_tile_variant(BASE_VARIANT)
    return binding


# ------------------------------------------------------------------ the benchmark configurations
def test_config1_gae_8x128(oracle, W, B):
    compare_all(oracle, W.config1(), algos=("gae",))


def test_config2_all_seven_4096x64(oracle, W, B):
    compare_all(oracle, W.config2())


@pytest.mark.parametrize("T", [32, 64, 128, 256, 512, 1024])
@pytest.mark.parametrize("with_truncs", [False, True])
def test_config3_sweep(oracle, W, B, T, with_truncs):
    ro = W.config3(T, with_truncs)
    compare_all(oracle, ro, algos=("gae", "vtrace"), use_truncs=with_truncs)


def test_config4_long_rows(oracle, W, B):
    ro = W.config4()
    gpu, ref, _ = compare_all(oracle, ro, algos=("gae", "discounted_return"), use_truncs=False)
    # gamma = 1 and rewards only at segment ends: adding zeros is exact in any association, so the
    # GPU returns must equal the oracle's bit for bit (after rounding the oracle to fp32).
    assert np.array_equal(gpu["discounted_return"], ref["discounted_return"].astype(np.float32))


def test_config5_full_size_all_seven(oracle, W, B):
    """16384 x 2048, truncation handling on: every element of every output against the oracle."""
    ro = W.config5()
    dev = Dev(ro)
    for a in ALL_ALGOS:                       # one algorithm at a time keeps host memory bounded
        gpu = run_gpu(dev, (a,))
        ref = run_oracle(oracle, ro, (a,))
        if isinstance(ref[a], tuple):
            for i, (g, r) in enumerate(zip(gpu[a], ref[a])):
                assert_close(f"{a}[{i}]", g, r)
        else:
            assert_close(a, gpu[a], ref[a])


def test_config5_full_size_extension_entry_points(oracle, W, B):
    """The entry points beyond the paper's API at the bench's full size, 16384 x 2048 with truncations,
    in the configuration bench.py times: time-major (all seven), bfloat16 GAE, skip-masked GAE.  Rows are
    independent, so the oracle checks every element of 192 sampled rows (first, last, and a seeded draw)."""
    import torch
    ro = W.config5()
    p = ro.params
    N, T = ro.N, ro.T
    rng = np.random.default_rng(5)
    rows = np.unique(np.concatenate([[0, 1, N - 2, N - 1], rng.integers(0, N, 188)]))
    sub = lambda a: None if a is None else np.ascontiguousarray(a[rows])
    import copy
    small = copy.copy(ro)
    for k in ("rewards", "values", "dones", "bootstrap", "truncs", "trunc_bootstrap", "q_sa", "expected_q", "log_rhos", "x"):
        setattr(small, k, sub(getattr(ro, k)))
    small.N = len(rows)
    ref = run_oracle(oracle, small, ALL_ALGOS)
    # time-major, all seven
    r, v, d, tr, bv = _tm(ro.rewards), _tm(ro.values), _tm(ro.dones), _tm(ro.truncs), _tm(ro.trunc_bootstrap)
    bt = guarded_upload(ro.bootstrap)
    take = lambda t: np.ascontiguousarray(t[:, guarded_upload(rows)].cpu().numpy().T)
    adv, ret = B.rlcs_gae_time_major(r, v, d, tr, bv, bt, gamma=p["gamma"], lam=p["lam"])
    assert_close("tm gae", take(adv), ref["gae"][0]); assert_close("tm ret", take(ret), ref["gae"][1])
    del adv, ret
    out = B.rlcs_td_lambda_time_major(r, v, d, tr, bv, bt, gamma=p["gamma"], lam=p["lam"])
    assert_close("tm td", take(out), ref["td_lambda"])
    out = B.rlcs_discounted_return_time_major(r, d, tr, bv, bt, gamma=p["gamma"])
    assert_close("tm disc", take(out), ref["discounted_return"])
    lr = _tm(ro.log_rhos)
    vs, pg = B.rlcs_vtrace_time_major(r, v, lr, d, tr, bv, bt, gamma=p["gamma"], rho_bar=p["rho_bar"], c_bar=p["c_bar"])
    assert_close("tm vs", take(vs), ref["vtrace"][0]); assert_close("tm pg", take(pg), ref["vtrace"][1])
    del vs, pg, v
    q, eq = _tm(ro.q_sa), _tm(ro.expected_q)
    out = B.rlcs_retrace_time_major(r, q, eq, lr, d, tr, bv, bt, gamma=p["gamma"], lam=p["lam"], c_bar=p["c_bar"])
    assert_close("tm retrace", take(out), ref["retrace"])
    del q, eq, lr, r, tr, bv, d
    x, dany = _tm(ro.x), _tm(ro.any_done)
    assert_close("tm elig", take(B.rlcs_elig_trace_time_major(x, dany, gamma=p["gamma"], lam=p["lam"])), ref["elig_trace"])
    assert_close("tm prefix", take(B.rlcs_episodic_prefix_sum_time_major(x, dany)), ref["prefix_ends_at"])
    del x, dany, out
    torch.cuda.empty_cache()
    # skip-masked GAE (row-major)
    dev = Dev(ro)
    skip = (np.random.default_rng(6).random((N, T)) < 0.3).astype(np.uint8)
    ws = B.Workspace(N, T)
    a, rt, fil = B.rlcs_gae_skip(dev.rewards, dev.values, dev.dones, dev.truncs, dev.trunc_bootstrap, dev.bootstrap,
                                 skip=guarded_upload(skip), gamma=p["gamma"], lam=p["lam"], workspace=ws)
    ra, rr, rf = oracle.gae_skip(small.rewards, small.values, small.dones, small.truncs, small.trunc_bootstrap, small.bootstrap,
                                 skip=np.ascontiguousarray(skip[rows]), gamma=p["gamma"], lam=p["lam"])
    pick = lambda t: t[guarded_upload(rows)].cpu().numpy()
    assert ws.device_status() == 0
    assert_close("skip adv", pick(a), ra); assert_close("skip ret", pick(rt), rr)
    assert np.array_equal(pick(fil).astype(np.float64), rf)


# ------------------------------------------------------------------ shape / flag matrix
SHAPES = [(1, 1), (3, 1), (1, 2), (2, 3), (3, 4), (8, 5), (3, 7), (64, 8), (3, 9), (8, 31), (64, 32), (3, 33),
          (8, 63), (2, 65), (3, 127), (8, 1000), (3, 2047), (2, 2048), (3, 2049), (2, 4097), (1, 20000)]


@pytest.mark.parametrize("N,T", SHAPES)
@pytest.mark.parametrize("p_flag", [0.0, 0.01, 0.5, 1.0])
def test_shape_matrix(oracle, W, B, N, T, p_flag):
    ro = W.make_rollout(90, N, T, p_done=p_flag, p_trunc=p_flag / 2, salt=N * 100003 + T)
    compare_all(oracle, ro)


@pytest.mark.parametrize("variant", [-1, 0, 5, 6, 19])
@pytest.mark.parametrize("N,T", [(37, 1000), (9, 2000), (130, 500), (64, 250), (301, 200), (1000, 100), (3, 1800), (700, 96)])
def test_row_aligned_tiles_and_look_back_agree(oracle, W, B, variant, N, T):
    """Rows shorter than a tile that do not divide it: with row-aligned tiling (a block takes a whole
    number of rows, its last threads idle) and without it (fixed tiles, carry through the workspace)
    the results match the oracle, and each other to rounding."""
    ro = W.make_rollout(93, N, T, p_done=0.004, p_trunc=0.004, salt=T)
    B.rlcs_debug_set_tile_variant(variant)
    try:
        gpu_on, _, _ = compare_all(oracle, ro)
        B.rlcs_debug_allow_row_tiles(False)
        gpu_off, _, _ = compare_all(oracle, ro)
    finally:
        B.rlcs_debug_allow_row_tiles(True)
        B.rlcs_debug_set_tile_variant(BASE_VARIANT)
    for a in gpu_on:
        for x, y in zip(gpu_on[a] if isinstance(gpu_on[a], tuple) else (gpu_on[a],), gpu_off[a] if isinstance(gpu_off[a], tuple) else (gpu_off[a],)):
            np.testing.assert_allclose(x, y, rtol=1e-5, atol=1e-4)
    # unaligned pointers take the element-wise instantiation of the same tiling
    compare_all(oracle, ro, offset=1)


@pytest.mark.parametrize("variant", [-1, 0, 6, 19])
@pytest.mark.parametrize("N,T", [(7, 3008), (5, 4096), (3, 16384), (11, 6000), (2, 40000), (300, 2512), (6, 2064)])
def test_one_block_per_row_agrees_with_the_carry_between_blocks(oracle, W, B, variant, N, T):
    """Rows longer than a tile: one thread block walking the whole row (carry in a register) against
    the carries between blocks (cluster / look-back).  Both match the oracle, and each other to
    rounding; where the row kernel does not apply (T not a multiple of the steps per thread, or a
    mostly empty last tile) the hook changes nothing."""
    ro = W.make_rollout(94, N, T, p_done=0.001, p_trunc=0.001, salt=T)
    B.rlcs_debug_set_tile_variant(variant)
    try:
        B.rlcs_debug_set_row_blocks(1)
        gpu_on, _, _ = compare_all(oracle, ro)
        B.rlcs_debug_set_row_blocks(0)
        gpu_off, _, _ = compare_all(oracle, ro)
    finally:
        B.rlcs_debug_set_row_blocks(-1)
        B.rlcs_debug_set_tile_variant(BASE_VARIANT)
    for a in gpu_on:
        for x, y in zip(gpu_on[a] if isinstance(gpu_on[a], tuple) else (gpu_on[a],), gpu_off[a] if isinstance(gpu_off[a], tuple) else (gpu_off[a],)):
            np.testing.assert_allclose(x, y, rtol=1e-5, atol=1e-4)


def test_one_block_per_row_is_the_default_with_many_rows(oracle, W, B):
    """Enough rows to fill the GPU: the row kernel is what runs (no carry workspace is needed)."""
    if BASE_VARIANT >= 0:
        pytest.skip("about the library's own choice of tile shape")
    N, T = 1200, 2064                                     # 2048 + one chunk of 16: no tile shape is filled to 70 % by such rows
    assert B.lib().rlcs_gae_carry_bytes(N, T, 1, 1) > 0   # ... so these rows are carried between blocks
    assert B.lib().rlcs_gae_carry_bytes(1500, 4112, 1, 1) == 0      # 4112 = 5 tiles of 1024 at 80 %: the 1024-step shape is taken
    assert B.lib().rlcs_gae_carry_bytes(1200, 4112, 1, 1) > 0       # ... but not for a thin second wave (1184 blocks fit at once)
    N, T = 1200, 6000
    ro = W.make_rollout(95, N, T, p_done=0.0005, p_trunc=0.0005)
    assert B.lib().rlcs_gae_carry_bytes(N, T, 1, 1) == 0
    compare_all(oracle, ro, algos=("gae", "vtrace", "discounted_return", "elig_trace"), workspace=None)


@pytest.mark.parametrize("variant", list(range(21)))
@pytest.mark.parametrize("N,T", [(5, 700), (4097, 3), (2, 9000), (64, 513)])
def test_tile_variants(oracle, W, B, variant, N, T):
    if not B.rlcs_debug_variant_built(variant):
        pytest.skip("tile variant not in this build (python -m paper_2608_17641_b200.build --all-variants compiles it)")
    B.rlcs_debug_set_tile_variant(variant)
    try:
        ro = W.make_rollout(91, N, T, p_done=0.01, p_trunc=0.005, salt=T)
        compare_all(oracle, ro)
    finally:
        B.rlcs_debug_set_tile_variant(BASE_VARIANT)


def test_long_row_without_resets_multi_window_lookback(oracle, W, B):
    """T = 131073 with no flags: 65 tiles per row, so the look-back crosses its 32-record window."""
    ro = W.make_rollout(92, 3, 131073, p_done=0.0, p_trunc=0.0)
    ro.params["gamma"] = 1.0
    ro.params["lam"] = 1.0
    compare_all(oracle, ro, algos=("gae", "discounted_return", "elig_trace", "prefix_ends_at", "vtrace", "retrace"))
    B.rlcs_debug_set_tile_variant(1)          # 512-step tiles: 257 tiles per row
    try:
        compare_all(oracle, ro, algos=("gae", "prefix_ends_at"))
    finally:
        B.rlcs_debug_set_tile_variant(BASE_VARIANT)


def test_randomized_shapes_flags_and_options(oracle, W, B):
    """Seeded fuzz over shapes, flag densities, kernel variants, pointer offsets and NULL options."""
    rng = np.random.default_rng(20260817)
    n_variants = 21
    for case in range(60):
        N = int(rng.integers(1, 200))
        T = int(rng.choice([rng.integers(1, 40), rng.integers(40, 3000), rng.integers(3000, 12000)]))
        if N * T > 600_000:
            N = max(1, 600_000 // T)
        p_done = float(rng.choice([0.0, 0.001, 0.02, 0.3]))
        p_trunc = float(rng.choice([0.0, 0.005, 0.2]))
        ro = W.make_rollout(108, N, T, p_done=p_done, p_trunc=p_trunc, salt=case)
        ro.params.update(gamma=float(rng.choice([0.9, 0.99, 1.0])), lam=float(rng.choice([0.0, 0.5, 0.95, 1.0])),
                         rho_bar=float(rng.choice([0.5, 1.0, 2.0])), c_bar=float(rng.choice([0.5, 1.0])))
        variant = int(rng.choice([BASE_VARIANT, int(rng.integers(0, n_variants))]))
        if variant >= 0 and not B.rlcs_debug_variant_built(variant):
            variant = BASE_VARIANT
        B.rlcs_debug_set_tile_variant(variant)
        try:
            compare_all(oracle, ro, offset=int(rng.choice([0, 0, 0, 1, 4, 8])),
                        use_truncs=bool(rng.random() < 0.7), use_bootstrap=bool(rng.random() < 0.8))
        except AssertionError as e:
            raise AssertionError(f"case {case}: N={N} T={T} p_done={p_done} p_trunc={p_trunc} variant={variant}: {e}")
        finally:
            B.rlcs_debug_set_tile_variant(BASE_VARIANT)


# ------------------------------------------------------------------ boundary cases
def _forced(W, N=6, T=300, salt=0):
    ro = W.make_rollout(93, N, T, p_done=0.02, p_trunc=0.02, salt=salt)
    ro.dones[0, 0] = 1                        # flags at both ends
    ro.dones[0, -1] = 1
    ro.truncs[1, 0] = 1
    ro.truncs[1, -1] = 1                      # truncated last step
    ro.dones[2, 17] = ro.truncs[2, 17] = 1    # both flags on one step
    ro.dones[3, -1] = ro.truncs[3, -1] = 1
    ro.dones[4, :] = 0
    ro.truncs[4, :] = 0                       # a row without any flag
    return ro


def test_forced_boundary_flags(oracle, W, B):
    compare_all(oracle, _forced(W))


def test_null_bootstrap_and_null_truncs(oracle, W, B):
    ro = _forced(W, salt=1)
    compare_all(oracle, ro, algos=BACKWARD, use_bootstrap=False)
    compare_all(oracle, ro, algos=BACKWARD, use_truncs=False)
    compare_all(oracle, ro, algos=BACKWARD, use_truncs=False, use_bootstrap=False)


@pytest.mark.parametrize("offset", [1, 2, 3, 4])       # 4 floats = 16-byte but not 32-byte aligned
@pytest.mark.parametrize("N,T", [(5, 333), (3, 2048), (2, 5000)])
def test_unaligned_pointers_take_elementwise_path(oracle, W, B, offset, N, T):
    ro = W.make_rollout(94, N, T, salt=offset)
    compare_all(oracle, ro, offset=offset)


def test_optional_outputs_null(oracle, W, B):
    ro = W.make_rollout(95, 7, 500)
    dev = Dev(ro)
    ws = B.Workspace(ro.N, ro.T)
    p = ro.params
    adv = B.rlcs_gae(dev.rewards, dev.values, dev.dones, dev.truncs, dev.trunc_bootstrap, dev.bootstrap,
                     gamma=p["gamma"], lam=p["lam"], want_returns=False, workspace=ws)
    vs = B.rlcs_vtrace(dev.rewards, dev.values, dev.log_rhos, dev.dones, dev.truncs, dev.trunc_bootstrap,
                       dev.bootstrap, gamma=p["gamma"], want_advantages=False, workspace=ws)
    ref = run_oracle(oracle, ro, ("gae", "vtrace"))
    assert_close("adv", adv.cpu().numpy(), ref["gae"][0])
    assert_close("vs", vs.cpu().numpy(), ref["vtrace"][0])


def test_guard_bands_untouched(oracle, W, B):
    """Outputs sit between NaN canaries; nothing outside [N*T) may be written."""
    import torch
    N, T, pad = 5, 1001, 64
    ro = W.make_rollout(96, N, T)
    dev = Dev(ro)
    ws = B.Workspace(N, T)
    p = ro.params

    def guarded():
        flat = torch.full((N * T + 2 * pad,), float("nan"), device="cuda")
        return flat, flat[pad:pad + N * T].view(N, T)

    f1, adv = guarded()
    f2, ret = guarded()
    f3, z = guarded()
    B.rlcs_gae(dev.rewards, dev.values, dev.dones, dev.truncs, dev.trunc_bootstrap, dev.bootstrap, gamma=p["gamma"],
               lam=p["lam"], advantages=adv, returns=ret, workspace=ws)
    B.rlcs_elig_trace(dev.x, dev.any_done, gamma=p["gamma"], lam=p["lam"], traces=z, workspace=ws)
    torch.cuda.synchronize()
    for f in (f1, f2, f3):
        assert torch.isnan(f[:pad]).all() and torch.isnan(f[-pad:]).all()
        assert torch.isfinite(f[pad:-pad]).all()


def test_nonbinary_flag_bytes(oracle, W, B):
    ro = W.make_rollout(97, 4, 600, p_done=0.05, p_trunc=0.05)
    ro.dones = (ro.dones * np.uint8(0x80)).astype(np.uint8)
    ro.truncs = (ro.truncs * np.uint8(0x7f)).astype(np.uint8)
    compare_all(oracle, ro)


def test_large_problem_variants_with_carry(oracle, W, B):
    """Above 2^23 steps the library picks per-algorithm tile shapes (more blocks per SM, 16 steps per
    thread); T = 3000 makes rows straddle every one of them, so the inter-block carry runs too."""
    ro = W.make_rollout(106, 2900, 3000, p_done=0.002, p_trunc=0.002)
    assert ro.N * ro.T > 1 << 23
    B.rlcs_debug_set_row_blocks(0)              # (with many rows the default would be one thread block per row)
    try:
        for a in ("gae", "vtrace", "td_lambda", "discounted_return", "elig_trace", "episodic_prefix_sum"):
            info = B.rlcs_debug_variant_for(a, True, ro.N, ro.T)
            assert BASE_VARIANT != -1 or info["variant"] not in (0, 6), (a, info)
        compare_all(oracle, ro)
    finally:
        B.rlcs_debug_set_row_blocks(-1)
    # the default for this shape: an 8-step tile shape that splits rows of 3000 into whole chunks, one block per row
    if BASE_VARIANT == -1:
        info = B.rlcs_debug_variant_for("gae", True, ro.N, ro.T)
        assert info["steps_per_thread"] == 8, info
        compare_all(oracle, ro, workspace=None)


@pytest.mark.parametrize("N,T,variant", [(5, 4096, 0), (3, 16384, 0), (64, 2048, 6), (7, 8192, 6), (9, 3072, 6), (2, 16384, 5),
                                              (3, 4096, 19)])
def test_cluster_carry_for_rows_of_whole_tiles(oracle, W, B, N, T, variant):
    """Rows of exactly 2..8 tiles: one thread-block cluster per row, carry in distributed shared
    memory and no workspace.  Against the oracle and against the workspace look-back."""
    tile = B.rlcs_debug_tile_elems(variant)
    assert T % tile == 0 and 2 <= T // tile <= 8
    ro = W.make_rollout(109, N, T, p_done=0.0005, p_trunc=0.0005, salt=T)
    B.rlcs_debug_set_tile_variant(variant)
    try:
        gpu, ref, _ = compare_all(oracle, ro, workspace=None)          # no workspace needed on this path
        B.rlcs_debug_allow_cluster_carry(False)
        other = run_gpu(Dev(ro), ALL_ALGOS)
    finally:
        B.rlcs_debug_allow_cluster_carry(True)
        B.rlcs_debug_set_tile_variant(BASE_VARIANT)
    for a in ALL_ALGOS:
        pairs = zip(gpu[a], other[a]) if isinstance(gpu[a], tuple) else [(gpu[a], other[a])]
        for x, y in pairs:
            np.testing.assert_allclose(x, y, rtol=1e-5, atol=1e-5, err_msg=a)


def test_wide_index_path_gives_identical_results(oracle, W, B):
    """The 64-bit row/timestep arithmetic (for 2^32 steps and more) against the 32-bit one, bit for
    bit, on shapes whose T is and is not a power of two, in both kernels."""
    for N, T in [(37, 1000), (5, 4096), (700, 7)]:
        ro = W.make_rollout(107, N, T, salt=T)
        dev = Dev(ro)
        for variant in (BASE_VARIANT, 8):
            B.rlcs_debug_set_tile_variant(variant)
            try:
                narrow = run_gpu(dev, ALL_ALGOS)
                B.rlcs_debug_force_wide_index(True)
                wide = run_gpu(dev, ALL_ALGOS)
            finally:
                B.rlcs_debug_force_wide_index(False)
                B.rlcs_debug_set_tile_variant(BASE_VARIANT)
            for a in ALL_ALGOS:
                pairs = zip(narrow[a], wide[a]) if isinstance(narrow[a], tuple) else [(narrow[a], wide[a])]
                for x, y in pairs:
                    assert np.array_equal(x, y), (a, N, T, variant)
        compare_all(oracle, ro)


def test_gamma_lambda_extremes(oracle, W, B):
    for g, l in [(0.0, 0.5), (1.0, 1.0), (0.5, 0.0), (1.0, 0.0)]:
        ro = W.make_rollout(98, 6, 777, p_done=0.01, p_trunc=0.01)
        ro.params.update(gamma=g, lam=l)
        compare_all(oracle, ro)


def test_clip_thresholds(oracle, W, B):
    for rb, cb in [(0.0, 0.0), (0.5, 2.0), (float("inf"), float("inf")), (1.5, 0.0)]:
        ro = W.make_rollout(99, 6, 555)
        ro.params.update(rho_bar=rb, c_bar=cb)
        compare_all(oracle, ro, algos=("vtrace", "retrace"))


# ------------------------------------------------------------------ segmentation is exact
def test_severed_steps_equal_alpha_exactly(oracle, W, B):
    ro = W.make_rollout(100, 16, 3000, p_done=0.03, p_trunc=0.0, with_truncs=False)
    gpu = run_gpu(Dev(ro), ("gae", "discounted_return"), use_truncs=False)
    tm = ro.dones != 0
    assert np.array_equal(gpu["discounted_return"][tm], ro.rewards[tm])
    assert np.array_equal(gpu["gae"][0][tm], (ro.rewards - ro.values)[tm])


def test_segment_isolation_bitwise(oracle, W, B):
    """Overwriting everything after a terminated step leaves the outputs up to it bit-identical
    (backward scans); overwriting everything before it leaves the later outputs bit-identical
    (forward scans).  The cut at t = 5000 is inside a tile, rows span several tiles."""
    ro = W.make_rollout(101, 3, 9000, p_done=0.0, p_trunc=0.0)
    cut = 5000
    ro.dones[:, cut] = 1
    base = run_gpu(Dev(ro), ALL_ALGOS)
    ro2 = W.make_rollout(101, 3, 9000, p_done=0.0, p_trunc=0.0, salt=7)
    ro2.dones[:, cut] = 1
    for k in ("rewards", "values", "q_sa", "expected_q", "log_rhos", "x", "trunc_bootstrap"):
        a = getattr(ro, k).copy()
        getattr(ro2, k)[:, :cut + 1] = a[:, :cut + 1]
    other = run_gpu(Dev(ro2), BACKWARD)
    for a in BACKWARD:
        pairs = zip(base[a], other[a]) if isinstance(base[a], tuple) else [(base[a], other[a])]
        for g0, g1 in pairs:
            assert np.array_equal(g0[:, :cut + 1], g1[:, :cut + 1]), a
            assert not np.array_equal(g0[:, cut + 1:], g1[:, cut + 1:]), a
    ro3 = W.make_rollout(101, 3, 9000, p_done=0.0, p_trunc=0.0, salt=9)
    ro3.dones[:, cut] = 1
    ro3.x[:, cut + 1:] = ro.x[:, cut + 1:]
    fwd = run_gpu(Dev(ro3), ("elig_trace", "prefix_ends_at"))
    for a in ("elig_trace", "prefix_ends_at"):
        assert np.array_equal(base[a][:, cut + 1:], fwd[a][:, cut + 1:]), a
        assert not np.array_equal(base[a][:, :cut + 1], fwd[a][:, :cut + 1]), a


def test_bootstrap_only_reaches_last_open_segment(oracle, W, B):
    ro = W.make_rollout(102, 4, 5000, p_done=0.001, p_trunc=0.0)
    base = run_gpu(Dev(ro), BACKWARD)
    ro.bootstrap = ro.bootstrap + np.float32(3.0)
    other = run_gpu(Dev(ro), BACKWARD)
    for n in range(ro.N):
        flagged = np.flatnonzero(ro.dones[n])
        last_reset = flagged[-1] if len(flagged) else -1
        for a in BACKWARD:
            g0 = base[a][0] if isinstance(base[a], tuple) else base[a]
            g1 = other[a][0] if isinstance(other[a], tuple) else other[a]
            assert np.array_equal(g0[n, :last_reset + 1], g1[n, :last_reset + 1]), a


def test_run_to_run_bit_identical(oracle, W, B):
    ro = W.config4(N=16, T=16384)
    dev = Dev(ro)
    first = run_gpu(dev, ("gae", "discounted_return"), use_truncs=False)
    for _ in range(5):
        again = run_gpu(dev, ("gae", "discounted_return"), use_truncs=False)
        assert np.array_equal(first["discounted_return"], again["discounted_return"])
        assert np.array_equal(first["gae"][0], again["gae"][0]) and np.array_equal(first["gae"][1], again["gae"][1])


def test_workspace_reuse_across_algorithms_and_shapes(oracle, W, B):
    """One workspace, many calls of different entry points and shapes on one stream."""
    big = B.Workspace(64, 5000)
    for (N, T) in [(64, 5000), (3, 700), (64, 4999)]:
        ro = W.make_rollout(103, N, T, salt=T)
        compare_all(oracle, ro, workspace=big)


# ------------------------------------------------------------------ GAE + advantage normalisation
@pytest.mark.parametrize("N,T", [(1, 1), (3, 7), (8, 128), (37, 1000), (64, 4096), (4096, 64), (5000, 2048)])
@pytest.mark.parametrize("ddof", [0, 1])
def test_gae_normalized(oracle, W, B, N, T, ddof):
    ro = W.make_rollout(110, N, T, salt=T)
    dev = Dev(ro)
    p = ro.params
    ws = B.Workspace(N, T, nbytes=B.lib().rlcs_gae_normalized_workspace_bytes(N, T))
    for use_tr in (True, False):
        tr, bv = (dev.truncs, dev.trunc_bootstrap) if use_tr else (None, None)
        adv, ret = B.rlcs_gae_normalized(dev.rewards, dev.values, dev.dones, tr, bv, dev.bootstrap, gamma=p["gamma"],
                                         lam=p["lam"], eps=1e-8, ddof=ddof, workspace=ws)
        ref_adv, ref_ret = oracle.gae_normalized(ro.rewards, ro.values, ro.dones, ro.truncs if use_tr else None,
                                                 ro.trunc_bootstrap if use_tr else None, ro.bootstrap,
                                                 gamma=p["gamma"], lam=p["lam"], eps=1e-8, ddof=ddof)
        assert ws.device_status() == 0
        assert_close("normalised advantages", adv.cpu().numpy(), ref_adv)
        assert_close("returns", ret.cpu().numpy(), ref_ret)
    # deterministic: a second call gives the same bits
    adv2, _ = B.rlcs_gae_normalized(dev.rewards, dev.values, dev.dones, None, None, dev.bootstrap, gamma=p["gamma"],
                                    lam=p["lam"], eps=1e-8, ddof=ddof, workspace=ws)
    assert np.array_equal(adv2.cpu().numpy(), adv.cpu().numpy())


def test_gae_normalized_back_to_back_calls_share_nothing_stale(oracle, W, B):
    """Three calls queued without a host synchronisation in between, on the same workspace and the same
    output tensors, with rewards of very different mean and spread: every call must rescale with its own
    mean and 1/(std + eps) (the follow-up kernels are placed on the SMs while the kernel before them is
    still running, and all of them read the two words from the same address)."""
    N, T = 3000, 512
    ro = W.make_rollout(116, N, T)
    p = ro.params
    scales = ((1.0, 0.0), (10.0, 5.0), (0.1, -3.0))
    ws = B.Workspace(N, T, nbytes=B.lib().rlcs_gae_normalized_workspace_bytes(N, T))
    dev = Dev(ro)
    rewards = [guarded_upload((ro.rewards * a + b).astype(np.float32)) for a, b in scales]
    adv, ret = dev.empty_out(), dev.empty_out()
    kept = []
    for r in rewards:
        B.rlcs_gae_normalized(r, dev.values, dev.dones, dev.truncs, dev.trunc_bootstrap, dev.bootstrap, gamma=p["gamma"],
                              lam=p["lam"], eps=1e-8, ddof=1, advantages=adv, returns=ret, workspace=ws)
        kept.append(adv.clone())
    for (a, b), got in zip(scales, kept):
        ref_adv, _ = oracle.gae_normalized((ro.rewards * a + b).astype(np.float32), ro.values, ro.dones, ro.truncs,
                                           ro.trunc_bootstrap, ro.bootstrap, gamma=p["gamma"], lam=p["lam"], eps=1e-8, ddof=1)
        assert_close(f"normalised advantages, rewards * {a} + {b}", got.cpu().numpy(), ref_adv)


@pytest.mark.parametrize("N,T", [(5, 4096), (3, 8192), (2, 32768), (470, 4096)])
def test_gae_normalized_one_block_per_row(oracle, W, B, N, T):
    """Rows of whole tiles walked by one thread block each (forced for few rows; the library's own
    choice at 470 x 4096): the per-tile sums are numbered row by row, the reduction sees every one of
    them once.  Against the oracle and against the carry between blocks."""
    ro = W.make_rollout(117, N, T, p_done=0.002, p_trunc=0.002, salt=T)
    dev = Dev(ro)
    p = ro.params
    ws = B.Workspace(N, T, nbytes=B.lib().rlcs_gae_normalized_workspace_bytes(N, T))
    call = lambda: [o.cpu().numpy() for o in B.rlcs_gae_normalized(dev.rewards, dev.values, dev.dones, dev.truncs,
                                                                   dev.trunc_bootstrap, dev.bootstrap, gamma=p["gamma"],
                                                                   lam=p["lam"], eps=1e-8, ddof=1, workspace=ws)]
    B.rlcs_debug_set_row_blocks(0)
    try:
        other = call()
        B.rlcs_debug_set_row_blocks(1)
        rows = call()
    finally:
        B.rlcs_debug_set_row_blocks(-1)
    ref_adv, ref_ret = oracle.gae_normalized(ro.rewards, ro.values, ro.dones, ro.truncs, ro.trunc_bootstrap, ro.bootstrap,
                                             gamma=p["gamma"], lam=p["lam"], eps=1e-8, ddof=1)
    assert_close("normalised advantages, rows", rows[0], ref_adv)
    assert_close("returns, rows", rows[1], ref_ret)
    np.testing.assert_allclose(rows[0], other[0], rtol=2e-5, atol=2e-5)
    if N >= 470:
        assert np.array_equal(rows[0], call()[0])                            # the default for this shape


def test_gae_normalized_with_a_mean_far_from_zero(oracle, W, B):
    """Rewards ~ N(100, 0.1^2), small values, lambda = 0.1, no flags: every advantage is close to
    100 with a spread of about 0.1, so |mean| is a thousand times the standard deviation -- the case
    in which single-precision sums of squares (sum A^2 - mean * sum A) lose the variance."""
    N, T, g, lam = 64, 1000, 0.99, 0.1
    ro = W.make_rollout(113, N, T, p_done=0.0, p_trunc=0.0, gamma=g, lam=lam)
    ro.rewards = (100.0 + 0.1 * ro.rewards).astype(np.float32)
    ro.values = (0.01 * ro.values).astype(np.float32)
    dev = Dev(ro)
    ws = B.Workspace(N, T, nbytes=B.lib().rlcs_gae_normalized_workspace_bytes(N, T))
    for ddof in (0, 1):
        adv, _ = B.rlcs_gae_normalized(dev.rewards, dev.values, dev.dones, None, None, None, gamma=g, lam=lam,
                                       eps=1e-8, ddof=ddof, workspace=ws)
        raw, _ = B.rlcs_gae(dev.rewards, dev.values, dev.dones, None, None, None, gamma=g, lam=lam, workspace=B.Workspace(N, T))
        ref_adv, _ = oracle.gae_normalized(ro.rewards, ro.values, ro.dones, None, None, None, gamma=g, lam=lam, eps=1e-8, ddof=ddof)
        got = adv.cpu().numpy().astype(np.float64)
        assert np.isfinite(got).all()
        # against the fp64 statistics of the GPU's own raw advantages: what is left is the rounding of
        # the mean to fp32 (half an ulp of 100, divided by the spread) and of the rescale itself
        a = raw.cpu().numpy().astype(np.float64)
        mean, std = a.mean(), a.std(ddof=ddof)
        cond = np.abs(a).max() / std
        assert cond > 200, cond
        np.testing.assert_allclose(got, (a - mean) / (std + 1e-8), rtol=1e-5, atol=2e-4)
        # and against the oracle: an fp32 rounding error of A is magnified by 1/std in the normalised value
        err = np.abs(got - ref_adv)
        assert err.max() <= 1e-4 + 1e-5 * np.abs(ref_adv).max() + 8 * 6e-8 * cond, (err.max(), cond)


def test_gae_normalized_argument_checks(oracle, W, B):
    ro = W.make_rollout(111, 4, 100)
    dev = Dev(ro)
    for kw in (dict(eps=-1.0), dict(eps=float("nan")), dict(eps=float("inf")), dict(ddof=2)):
        with pytest.raises(B.RlcsError) as e:
            B.rlcs_gae_normalized(dev.rewards, dev.values, dev.dones, gamma=0.99, lam=0.95, **kw)
        assert e.value.status == B.RLCS_ERR_ARG
    small = B.Workspace(4, 100, nbytes=256)
    with pytest.raises(B.RlcsError) as e:
        B.rlcs_gae_normalized(dev.rewards, dev.values, dev.dones, gamma=0.99, lam=0.95, workspace=small)
    assert e.value.status == B.RLCS_ERR_WORKSPACE


# ------------------------------------------------------------------ Retrace from [N,T,A] tensors
def _probs_gpu(B, ro, q, pi, mu, act, use_truncs=True, use_bootstrap=True, offset=0):
    import torch
    dev = Dev(ro, offset=offset)

    up3 = lambda a: guarded_upload(a, offset)

    ws = B.Workspace(ro.N, ro.T)
    p = ro.params
    out = B.rlcs_retrace_probs(dev.rewards, up3(q), up3(pi), up3(mu), guarded_upload(act), dev.dones,
                               dev.truncs if use_truncs else None, dev.trunc_bootstrap if use_truncs else None,
                               dev.bootstrap if use_bootstrap else None, gamma=p["gamma"], lam=p["lam"], c_bar=p["c_bar"],
                               q_targets=dev.empty_out(), workspace=ws)
    torch.cuda.synchronize()
    assert ws.device_status() == 0
    return out.cpu().numpy()


@pytest.mark.parametrize("A", [1, 2, 3, 4, 5, 8, 16, 18])
@pytest.mark.parametrize("N,T", [(1, 1), (3, 7), (8, 128), (5, 1000), (2, 4096), (300, 257)])
def test_retrace_probs_matches_oracle(oracle, W, B, A, N, T):
    ro = W.make_rollout(112, N, T, p_done=0.02, p_trunc=0.01, salt=A)
    q, pi, mu, act = W.make_action_tensors(112, N, T, A, salt=T)
    for use_tr, use_bt in ((True, True), (False, True), (True, False)):
        got = _probs_gpu(B, ro, q, pi, mu, act, use_tr, use_bt)
        ref = oracle.retrace_probs(ro.rewards, q, pi, mu, act, ro.dones, ro.truncs if use_tr else None,
                                   ro.trunc_bootstrap if use_tr else None, ro.bootstrap if use_bt else None,
                                   gamma=ro.params["gamma"], lam=ro.params["lam"], c_bar=ro.params["c_bar"])
        assert_close(f"retrace_probs A={A}", got, ref)


def test_retrace_probs_unaligned_and_long_rows(oracle, W, B):
    """Pointers off 16-byte alignment (element-wise row reads), and T = 16384: the register need of the
    tile does not depend on T (the paper's kernel spilled from T = 4096 on)."""
    for (N, T, A, off) in [(4, 600, 4, 1), (3, 600, 8, 2), (2, 16384, 4, 0), (64, 16384, 4, 0)]:
        ro = W.make_rollout(113, N, T, p_done=0.001, p_trunc=0.001, salt=A)
        q, pi, mu, act = W.make_action_tensors(113, N, T, A, salt=off)
        got = _probs_gpu(B, ro, q, pi, mu, act, offset=off)
        ref = oracle.retrace_probs(ro.rewards, q, pi, mu, act, ro.dones, ro.truncs, ro.trunc_bootstrap, ro.bootstrap,
                                   gamma=ro.params["gamma"], lam=ro.params["lam"], c_bar=ro.params["c_bar"])
        assert_close(f"retrace_probs {N}x{T}x{A} offset {off}", got, ref)


@pytest.mark.parametrize("A", [3, 4, 8, 16])
@pytest.mark.parametrize("N,T", [(5, 2048), (3, 4096), (2, 16384), (470, 2048)])
def test_retrace_probs_one_block_per_row(oracle, W, B, A, N, T):
    """Rows of whole 1024-step tiles walked by one thread block each (forced here for few rows; the
    library's own choice from about three rows per SM, which 470 x 2048 reaches): against the oracle
    and against the carry through tile records."""
    ro = W.make_rollout(115, N, T, p_done=0.002, p_trunc=0.002, salt=A + T)
    q, pi, mu, act = W.make_action_tensors(115, N, T, A, salt=N)
    B.rlcs_debug_set_row_blocks(0)
    try:
        records = _probs_gpu(B, ro, q, pi, mu, act)
        B.rlcs_debug_set_row_blocks(1)
        rows = _probs_gpu(B, ro, q, pi, mu, act)
        rows_plain = _probs_gpu(B, ro, q, pi, mu, act, use_truncs=False, use_bootstrap=False)
    finally:
        B.rlcs_debug_set_row_blocks(-1)
    kw = dict(gamma=ro.params["gamma"], lam=ro.params["lam"], c_bar=ro.params["c_bar"])
    assert_close(f"retrace_probs rows {N}x{T}x{A}", rows,
                 oracle.retrace_probs(ro.rewards, q, pi, mu, act, ro.dones, ro.truncs, ro.trunc_bootstrap, ro.bootstrap, **kw))
    assert_close(f"retrace_probs rows, plain {N}x{T}x{A}", rows_plain,
                 oracle.retrace_probs(ro.rewards, q, pi, mu, act, ro.dones, None, None, None, **kw))
    np.testing.assert_allclose(rows, records, rtol=1e-5, atol=1e-5)
    if N >= 470:
        assert np.array_equal(rows, _probs_gpu(B, ro, q, pi, mu, act))      # the default for this shape


def test_retrace_probs_agrees_with_scalar_entry_point(oracle, W, B):
    """The tensor form and rlcs_retrace on inputs derived from the tensors (gather, dot, log) agree."""
    import torch
    N, T, A = 16, 3000, 4
    ro = W.make_rollout(114, N, T)
    q, pi, mu, act = W.make_action_tensors(114, N, T, A)
    got = _probs_gpu(B, ro, q, pi, mu, act)
    idx = act[..., None].astype(np.int64)
    ro.q_sa = np.take_along_axis(q, idx, axis=2)[..., 0].copy()
    ro.expected_q = np.einsum("nta,nta->nt", pi.astype(np.float64), q.astype(np.float64)).astype(np.float32)
    ro.log_rhos = np.log(np.take_along_axis(pi, idx, axis=2)[..., 0].astype(np.float64)
                         / np.take_along_axis(mu, idx, axis=2)[..., 0].astype(np.float64)).astype(np.float32)
    scalar = run_gpu(Dev(ro), ("retrace",))["retrace"]
    np.testing.assert_allclose(got, scalar, rtol=3e-5, atol=3e-5)


# ------------------------------------------------------------------ vector-valued eligibility traces
@pytest.mark.parametrize("N,T,D", [(1, 1, 1), (3, 7, 5), (8, 128, 64), (64, 257, 16), (4096, 40, 8), (2, 5000, 128),
                                    (3, 16384, 32), (1, 70000, 4), (5, 999, 3), (7, 300, 130),
                                    (64, 4096, 64), (100, 3000, 32), (48, 2000, 96), (60, 1000, 36)])
def test_vector_eligibility_trace(oracle, W, B, N, T, D):
    import torch
    rng = np.random.default_rng(N * 7919 + T * 31 + D)
    x = rng.standard_normal((N, T, D)).astype(np.float32)
    d = (rng.random((N, T)) < 0.02).astype(np.uint8)
    d[:, 0] = rng.integers(0, 2, N)                      # a flag on the very first step
    xd, dd = guarded_upload(x), guarded_upload(d)
    ref = oracle.elig_trace_vec(x, d, gamma=0.99, lam=0.95)
    got = B.rlcs_elig_trace_vec(xd, dd, gamma=0.99, lam=0.95).cpu().numpy()
    assert_close(f"vector trace {N}x{T}x{D}", got, ref)
    again = B.rlcs_elig_trace_vec(xd, dd, gamma=0.99, lam=0.95).cpu().numpy()
    assert np.array_equal(got, again)
    # pointer off 16-byte alignment: element-wise variant
    xo = guarded_upload(x, 1)
    got1 = B.rlcs_elig_trace_vec(xo, dd, gamma=0.99, lam=0.95).cpu().numpy()
    assert_close("vector trace, unaligned", got1, ref)
    # against the scalar entry point, component by component
    if N * T * D <= 200_000:
        for c in range(min(D, 3)):
            sc = B.rlcs_elig_trace(xd[:, :, c].contiguous(), dd, gamma=0.99, lam=0.95, workspace=B.Workspace(N, T))
            np.testing.assert_allclose(got[:, :, c], sc.cpu().numpy(), rtol=1e-5, atol=1e-5)


def test_vector_trace_argument_checks(oracle, W, B):
    L = B.lib()
    P = 0x7f0000000000
    assert L.rlcs_elig_trace_vec(P, P, P, 4, 8, 0, 0.9, 0.9, None, 0, None) == B.RLCS_OK
    assert L.rlcs_elig_trace_vec(P, P, P, 4, 8, -1, 0.9, 0.9, None, 0, None) == B.RLCS_ERR_SIZE
    assert L.rlcs_elig_trace_vec(None, P, P, 4, 8, 4, 0.9, 0.9, None, 0, None) == B.RLCS_ERR_NULL
    assert L.rlcs_elig_trace_vec(P, P, P, 4, 8, 4, 1.5, 0.9, None, 0, None) == B.RLCS_ERR_ARG
    assert L.rlcs_elig_trace_vec(P + 2, P, P, 4, 8, 4, 0.9, 0.9, None, 0, None) == B.RLCS_ERR_ALIGN
    need = L.rlcs_elig_trace_vec_workspace_bytes(2, 100000, 8)
    assert need > 0 and L.rlcs_elig_trace_vec_workspace_bytes(100000, 64, 64) == 0
    assert L.rlcs_elig_trace_vec(P, P, P, 2, 100000, 8, 0.9, 0.9, None, 0, None) == B.RLCS_ERR_WORKSPACE


@pytest.mark.parametrize("N,T,D", [(1, 1, 1), (3, 7, 5), (8, 128, 64), (64, 257, 16), (4096, 40, 8), (2, 5000, 128),
                                    (3, 16384, 32), (5, 999, 3), (64, 4096, 64), (100, 3000, 32), (48, 2000, 96), (60, 1000, 36)])
def test_per_dimension_beta_eligibility_trace(oracle, W, B, N, T, D):
    import torch
    rng = np.random.default_rng(N * 7919 + T * 31 + D + 1)
    x = rng.standard_normal((N, T, D)).astype(np.float32)
    beta = rng.uniform(0.5, 1.0, (N, T, D)).astype(np.float32)
    d = (rng.random((N, T)) < 0.02).astype(np.uint8)
    d[:, 0] = rng.integers(0, 2, N)
    xd, bd, dd = guarded_upload(x), guarded_upload(beta), guarded_upload(d)
    ref = oracle.elig_trace_vec_beta(x, beta, d)
    got = B.rlcs_elig_trace_vec_beta(xd, bd, dd).cpu().numpy()
    assert_close(f"per-dimension trace {N}x{T}x{D}", got, ref)
    # pointers off 16-byte alignment: element-wise variant
    off = lambda t: torch.cat([t.new_zeros(1), t.reshape(-1)])[1:].view(t.shape)
    got1 = B.rlcs_elig_trace_vec_beta(off(xd), off(bd), dd).cpu().numpy()
    assert_close("per-dimension trace, unaligned", got1, ref)
    # a constant beta is the shared-scalar entry point: bit for bit when both walk whole rows with one
    # thread per component group (same FMA per step), to rounding under the planned kernels
    const = torch.full_like(xd, 0.25)
    same = B.rlcs_elig_trace_vec_beta(xd, const, dd)
    scalar = B.rlcs_elig_trace_vec(xd, dd, gamma=0.5, lam=0.5)
    assert_close("constant beta vs shared decay", same.cpu().numpy(), scalar.cpu().numpy().astype(np.float64))
    B.rlcs_debug_vec_trace_plan(8, 1)
    try:
        assert torch.equal(B.rlcs_elig_trace_vec_beta(xd, const, dd), B.rlcs_elig_trace_vec(xd, dd, gamma=0.5, lam=0.5))
    finally:
        B.rlcs_debug_vec_trace_plan(0, 0)


@pytest.mark.parametrize("plan", [(1, 0), (8, 1), (16, 1), (32, 1), (8, 3), (32, 2), (16, 7), "chained", "unchained"])
@pytest.mark.parametrize("N,T,D", [(8, 128, 64), (5, 999, 3), (48, 2000, 96), (3, 700, 36), (130, 300, 32)])
def test_vector_trace_plans_agree(oracle, W, B, N, T, D, plan):
    """Every load-ahead depth, forced time cuts and the block kernel give the oracle's traces."""
    import torch
    rng = np.random.default_rng(N * 7919 + T * 31 + D + 2)
    x = rng.standard_normal((N, T, D)).astype(np.float32)
    beta = rng.uniform(0.5, 1.0, (N, T, D)).astype(np.float32)
    d = (rng.random((N, T)) < 0.02).astype(np.uint8)
    xd, bd, dd = guarded_upload(x), guarded_upload(beta), guarded_upload(d)
    if isinstance(plan, str):            # the block kernel, its time axis always / never cut into chained chunks
        B.rlcs_debug_vec_trace_plan(1, 0)
        B.rlcs_debug_time_major_path(5 if plan == "chained" else 4)
    else:
        B.rlcs_debug_vec_trace_plan(*plan)
    try:
        got = B.rlcs_elig_trace_vec(xd, dd, gamma=0.99, lam=0.95).cpu().numpy()
        gotb = B.rlcs_elig_trace_vec_beta(xd, bd, dd).cpu().numpy()
        if plan == "chained":
            assert np.array_equal(gotb, B.rlcs_elig_trace_vec_beta(xd, bd, dd).cpu().numpy())
    finally:
        B.rlcs_debug_vec_trace_plan(0, 0)
        B.rlcs_debug_time_major_path(0)
    assert_close(f"vector trace, plan {plan}", got, oracle.elig_trace_vec(x, d, gamma=0.99, lam=0.95))
    assert_close(f"per-dimension trace, plan {plan}", gotb, oracle.elig_trace_vec_beta(x, beta, d))


@pytest.mark.parametrize("p_flag", [0.0, 0.004, 0.02, 0.5])
@pytest.mark.parametrize("N,T,D", [(3, 2100, 64), (2, 1024, 36), (5, 777, 128)])
def test_vector_trace_chained_kernel_single_walk(oracle, W, B, N, T, D, p_flag):
    """The chained kernel of the vector traces walks a chunk once and finishes the steps before the
    chunk's first cut when the carry arrives: no cut at all (every step of every later chunk waits for
    its carry), rare cuts, the recipe's rate, every other step cut, and cuts placed on the steps around
    the chunk boundaries (256 steps with the shared decay, 128 with a decay tensor); the last chunk is
    ragged.  gamma * lambda = 1 carries a chunk's value undamped through all later chunks."""
    rng = np.random.default_rng(N * 131 + T * 7 + D + int(p_flag * 1000))
    x = rng.standard_normal((N, T, D)).astype(np.float32)
    beta = rng.uniform(0.5, 1.0, (N, T, D)).astype(np.float32)
    d = (rng.random((N, T)) < p_flag).astype(np.uint8)
    if p_flag > 0:
        for t in (126, 127, 128, 255, 256, 257, 511, 512, 768):
            if t < T:
                d[t % N, t] = 1
    xd, bd, dd = guarded_upload(x), guarded_upload(beta), guarded_upload(d)
    B.rlcs_debug_vec_trace_plan(1, 0)
    B.rlcs_debug_time_major_path(5)
    try:
        got = B.rlcs_elig_trace_vec(xd, dd, gamma=0.99, lam=0.95).cpu().numpy()
        got1 = B.rlcs_elig_trace_vec(xd, dd, gamma=1.0, lam=1.0).cpu().numpy()
        gotb = B.rlcs_elig_trace_vec_beta(xd, bd, dd).cpu().numpy()
        assert np.array_equal(got, B.rlcs_elig_trace_vec(xd, dd, gamma=0.99, lam=0.95).cpu().numpy())
    finally:
        B.rlcs_debug_vec_trace_plan(0, 0)
        B.rlcs_debug_time_major_path(0)
    assert_close("vector trace, chained", got, oracle.elig_trace_vec(x, d, gamma=0.99, lam=0.95))
    assert_close("vector trace, chained, undamped", got1, oracle.elig_trace_vec(x, d, gamma=1.0, lam=1.0))
    assert_close("per-dimension trace, chained", gotb, oracle.elig_trace_vec_beta(x, beta, d))


def test_vector_trace_chained_wait_runs_out_and_reports_timeout(oracle, W, B):
    """The single-walk chained kernel with one block that never publishes its chunk and no cut
    anywhere (every later chunk of that chain needs a carry): the waits run out of polls, the kernel
    finishes, the status word says TIMEOUT, and the next call on the workspace is right."""
    import torch
    N, T, D = 4, 4096, 64
    rng = np.random.default_rng(4711)
    x = rng.standard_normal((N, T, D)).astype(np.float32)
    d = np.zeros((N, T), np.uint8)
    xd, dd = guarded_upload(x), guarded_upload(d)
    B.rlcs_debug_vec_trace_plan(1, 0)
    B.rlcs_debug_time_major_path(5)
    try:
        ws = B.Workspace(N, T, nbytes=int(B.lib().rlcs_elig_trace_vec_workspace_bytes(N, T, D)))
        B.rlcs_debug_set_carry_fault(2, 50)
        try:
            B.rlcs_elig_trace_vec(xd, dd, gamma=0.99, lam=0.95, workspace=ws)
            torch.cuda.synchronize()
            assert ws.device_status() == B.RLCS_ERR_TIMEOUT
        finally:
            B.rlcs_debug_set_carry_fault(-1, 0)
        assert ws.device_status() == B.RLCS_OK
        got = B.rlcs_elig_trace_vec(xd, dd, gamma=0.99, lam=0.95, workspace=ws).cpu().numpy()
        assert ws.device_status() == B.RLCS_OK
    finally:
        B.rlcs_debug_vec_trace_plan(0, 0)
        B.rlcs_debug_time_major_path(0)
    assert_close("vector trace after the timeout", got, oracle.elig_trace_vec(x, d, gamma=0.99, lam=0.95))


def test_per_dimension_beta_argument_checks(oracle, W, B):
    L = B.lib()
    P = 0x7f0000000000
    assert L.rlcs_elig_trace_vec_beta(P, P, P, P, 4, 8, 0, None, 0, None) == B.RLCS_OK
    assert L.rlcs_elig_trace_vec_beta(P, None, P, P, 4, 8, 4, None, 0, None) == B.RLCS_ERR_NULL
    assert L.rlcs_elig_trace_vec_beta(P, P + 2, P, P, 4, 8, 4, None, 0, None) == B.RLCS_ERR_ALIGN
    assert L.rlcs_elig_trace_vec_beta_workspace_bytes(2, 100000, 8) > L.rlcs_elig_trace_vec_workspace_bytes(2, 100000, 8)
    assert L.rlcs_elig_trace_vec_beta(P, P, P, P, 2, 100000, 8, None, 0, None) == B.RLCS_ERR_WORKSPACE


# ------------------------------------------------------------------ observation-skip masking
def _skip_case(W, N, T, p_skip, p_flag, salt=0):
    ro = W.make_rollout(130, N, T, p_done=p_flag, p_trunc=p_flag / 2, salt=salt + T)
    rng = np.random.default_rng(N * 31 + T + salt)
    skip = (rng.random((N, T)) < p_skip).astype(np.uint8)
    # observation tokens come in runs: lengthen every masked step into a short span
    for k in (1, 2):
        skip[:, k:] |= skip[:, :-k] & (rng.random((N, T - k)) < 0.6).astype(np.uint8) if T > k else 0
    return ro, skip


@pytest.mark.parametrize("N,T", [(1, 1), (3, 7), (5, 1001), (64, 512), (4096, 64), (7, 5000), (2, 40000), (4, 2048)])
@pytest.mark.parametrize("p_skip,p_flag", [(0.0, 0.02), (0.2, 0.0), (0.2, 0.02), (0.9, 0.05), (1.0, 0.0)])
def test_gae_with_observation_skip_masking(oracle, W, B, N, T, p_skip, p_flag):
    """Flags may sit on masked steps as well: the oracle defines that case too."""
    import torch
    ro, skip = _skip_case(W, N, T, p_skip, p_flag)
    p = ro.params
    dev = Dev(ro)
    sk = guarded_upload(skip)
    ws = B.Workspace(N, T)
    adv, ret, fil = B.rlcs_gae_skip(dev.rewards, dev.values, dev.dones, dev.truncs, dev.trunc_bootstrap, dev.bootstrap,
                                    skip=sk, gamma=p["gamma"], lam=p["lam"], workspace=ws)
    torch.cuda.synchronize()
    assert ws.device_status() == 0
    ra, rr, rf = oracle.gae_skip(ro.rewards, ro.values, ro.dones, ro.truncs, ro.trunc_bootstrap, ro.bootstrap, skip=skip,
                                 gamma=p["gamma"], lam=p["lam"])
    assert np.array_equal(fil.cpu().numpy().astype(np.float64), rf)          # W is copied, never computed
    assert_close("skip adv", adv.cpu().numpy(), ra)
    assert_close("skip ret", ret.cpu().numpy(), rr)
    if p_skip == 0.0:                                                        # nothing masked: rlcs_gae, bit for bit on the same tile shape
        B.rlcs_debug_set_tile_variant(0)
        try:
            a0, _ = B.rlcs_gae(dev.rewards, dev.values, dev.dones, dev.truncs, dev.trunc_bootstrap, dev.bootstrap,
                               gamma=p["gamma"], lam=p["lam"], workspace=ws)
            a1, _, _ = B.rlcs_gae_skip(dev.rewards, dev.values, dev.dones, dev.truncs, dev.trunc_bootstrap, dev.bootstrap,
                                       skip=sk, gamma=p["gamma"], lam=p["lam"], workspace=ws)
        finally:
            B.rlcs_debug_set_tile_variant(BASE_VARIANT)
        assert torch.equal(a0, a1)


@pytest.mark.parametrize("p_skip,p_flag", [(0.3, 0.002), (0.9, 0.0), (0.0, 0.02)])
@pytest.mark.parametrize("N,T", [(5, 4096), (3, 8192), (2, 16384), (470, 4096)])
def test_gae_skip_one_block_per_row(oracle, W, B, N, T, p_skip, p_flag):
    """Rows of whole 2048-step tiles walked by one thread block each, both carries (filled value and
    advantage) in registers -- forced here for few rows; the library's own choice from about three rows
    per SM, which 470 x 4096 reaches: against the oracle and against the carry through tile records,
    with and without truncation tensors."""
    import torch
    ro, skip = _skip_case(W, N, T, p_skip, p_flag, salt=3)
    p = ro.params
    dev = Dev(ro)
    sk = guarded_upload(skip)
    ws = B.Workspace(N, T)

    def call(use_tr=True):
        tr, bv = (dev.truncs, dev.trunc_bootstrap) if use_tr else (None, None)
        out = B.rlcs_gae_skip(dev.rewards, dev.values, dev.dones, tr, bv, dev.bootstrap, skip=sk, gamma=p["gamma"],
                              lam=p["lam"], workspace=ws)
        torch.cuda.synchronize()
        assert ws.device_status() == 0
        return [o.cpu().numpy() for o in out]

    B.rlcs_debug_set_row_blocks(0)
    try:
        records = call()
        B.rlcs_debug_set_row_blocks(1)
        rows = call()
        rows_plain = call(use_tr=False)
    finally:
        B.rlcs_debug_set_row_blocks(-1)
    ra, rr, rf = oracle.gae_skip(ro.rewards, ro.values, ro.dones, ro.truncs, ro.trunc_bootstrap, ro.bootstrap, skip=skip,
                                 gamma=p["gamma"], lam=p["lam"])
    assert np.array_equal(rows[2].astype(np.float64), rf)
    assert_close("skip adv, rows", rows[0], ra)
    assert_close("skip ret, rows", rows[1], rr)
    pa, pr, pf = oracle.gae_skip(ro.rewards, ro.values, ro.dones, None, None, ro.bootstrap, skip=skip, gamma=p["gamma"],
                                 lam=p["lam"])
    assert np.array_equal(rows_plain[2].astype(np.float64), pf)
    assert_close("skip adv, rows, no truncation tensors", rows_plain[0], pa)
    assert_close("skip ret, rows, no truncation tensors", rows_plain[1], pr)
    for x, y in zip(rows, records):
        np.testing.assert_allclose(x, y, rtol=1e-5, atol=1e-5)
    if N >= 470:
        for x, y in zip(rows, call()):                                       # the default for this shape
            assert np.array_equal(x, y)


def test_gae_skip_options_alignment_and_large_problem(oracle, W, B):
    import torch
    # no truncation tensors, no bootstrap, no returns; pointers off 16-byte alignment
    ro, skip = _skip_case(W, 6, 900, 0.3, 0.03, salt=1)
    p = ro.params
    for offset in (0, 1):
        dev = Dev(ro, offset=offset)
        sk = guarded_upload(skip, offset)
        adv, fil = B.rlcs_gae_skip(dev.rewards, dev.values, dev.dones, skip=sk, gamma=p["gamma"], lam=p["lam"],
                                   values_filled=dev.empty_out(), advantages=dev.empty_out(), want_returns=False,
                                   workspace=B.Workspace(ro.N, ro.T))
        ra, _, rf = oracle.gae_skip(ro.rewards, ro.values, ro.dones, skip=skip, gamma=p["gamma"], lam=p["lam"])
        assert_close(f"skip adv, offset {offset}", adv.cpu().numpy(), ra)
        assert np.array_equal(fil.cpu().numpy().astype(np.float64), rf)
    # above 2^23 steps (per-algorithm tile shapes), rows straddling tiles: look-back carries both scans
    ro, skip = _skip_case(W, 2900, 3000, 0.3, 0.002, salt=2)
    p = ro.params
    dev = Dev(ro)
    ws = B.Workspace(ro.N, ro.T)
    adv, ret, fil = B.rlcs_gae_skip(dev.rewards, dev.values, dev.dones, dev.truncs, dev.trunc_bootstrap, dev.bootstrap,
                                    skip=guarded_upload(skip), gamma=p["gamma"], lam=p["lam"], workspace=ws)
    ra, rr, rf = oracle.run_rows_parallel(
        lambda **k: oracle.gae_skip(k["rewards"], k["values"], k["dones"], k["truncs"], k["trunc_bootstrap"], k["bootstrap"],
                                    skip=k["skip"], gamma=p["gamma"], lam=p["lam"]),
        dict(rewards=ro.rewards, values=ro.values, dones=ro.dones, truncs=ro.truncs, trunc_bootstrap=ro.trunc_bootstrap,
             skip=skip), dict(bootstrap=ro.bootstrap), 8)
    assert ws.device_status() == 0
    assert_close("skip adv, large", adv.cpu().numpy(), ra)
    assert_close("skip ret, large", ret.cpu().numpy(), rr)
    assert np.array_equal(fil.cpu().numpy().astype(np.float64), rf)
    # argument checks
    L = B.lib()
    P = 0x7f0000000000
    g = lambda **k: L.rlcs_gae_skip(P, P, P, None, None, None, k.get("sk", P), k.get("fil", P), P, None, k.get("N", 4), 128,
                                    k.get("g", 0.9), 0.9, None, 0, None)
    assert g(N=0) == B.RLCS_OK and g(sk=None) == B.RLCS_ERR_NULL and g(fil=None) == B.RLCS_ERR_NULL
    assert g(g=1.5) == B.RLCS_ERR_ARG and g(fil=P + 2) == B.RLCS_ERR_ALIGN


# ------------------------------------------------------------------ time-major [T, N] entry points
def _tm(a):
    import torch
    return None if a is None else guarded_upload(np.ascontiguousarray(np.asarray(a).T))


@pytest.fixture
def tm_path(B, request):
    B.rlcs_debug_time_major_path(request.param)
    yield request.param
    B.rlcs_debug_time_major_path(0)


@pytest.mark.parametrize("N,T", [(1, 1), (3, 7), (8, 128), (300, 65), (4096, 64), (64, 3000), (5, 20000), (40000, 33),
                                 (16, 1), (48, 517), (4112, 70), (16, 20000), (20000, 9), (19024, 300)])
@pytest.mark.parametrize("p_flag", [0.0, 0.02, 0.5])
@pytest.mark.parametrize("tm_path", [1, 2, 3, 4, 5], indirect=True)
def test_time_major_entry_points(oracle, W, B, N, T, p_flag, tm_path):
    """All seven algorithms on [T, N] tensors against the oracle run on the transposed arrays; shapes
    cover the single-pass walk (many environments), the cut time axis (few environments), both
    kernels (register walk; shared-memory ring, which needs N % 16 == 0, with two columns per lane
    where the library uses them -- GAE and TD(lambda) without truncations from 18944 environments up
    -- and with one column per lane) and ragged last warps."""
    if tm_path != 1 and N % 16 != 0:
        pytest.skip("the ring needs N % 16 == 0; the register walk is covered by tm_path = 1")
    if tm_path == 3 and N < 18944:
        pytest.skip("one column per lane is what tm_path = 2 already takes at this size")
    if tm_path == 4 and (N >= 3072 or T <= 64):
        pytest.skip("the time axis is not cut at this size: three launches against one chained launch is no choice here")
    if tm_path == 5 and T <= 64:
        pytest.skip("no chunk of the chained kernel is shorter than the whole window")
    ro = W.make_rollout(115, N, T, p_done=p_flag, p_trunc=p_flag / 2, salt=T)
    p = ro.params
    ref = run_oracle(oracle, ro, ALL_ALGOS)
    r, v, d, tr, bv = _tm(ro.rewards), _tm(ro.values), _tm(ro.dones), _tm(ro.truncs), _tm(ro.trunc_bootstrap)
    q, eq, lr, x, dany = _tm(ro.q_sa), _tm(ro.expected_q), _tm(ro.log_rhos), _tm(ro.x), _tm(ro.any_done)
    import torch
    bt = guarded_upload(ro.bootstrap)
    back = lambda t: t.cpu().numpy().T
    adv, ret = B.rlcs_gae_time_major(r, v, d, tr, bv, bt, gamma=p["gamma"], lam=p["lam"])
    assert_close("gae adv", np.ascontiguousarray(back(adv)), ref["gae"][0])
    assert_close("gae ret", np.ascontiguousarray(back(ret)), ref["gae"][1])
    vs, pg = B.rlcs_vtrace_time_major(r, v, lr, d, tr, bv, bt, gamma=p["gamma"], rho_bar=p["rho_bar"], c_bar=p["c_bar"])
    assert_close("vtrace vs", np.ascontiguousarray(back(vs)), ref["vtrace"][0])
    assert_close("vtrace adv", np.ascontiguousarray(back(pg)), ref["vtrace"][1])
    out = B.rlcs_retrace_time_major(r, q, eq, lr, d, tr, bv, bt, gamma=p["gamma"], lam=p["lam"], c_bar=p["c_bar"])
    assert_close("retrace", np.ascontiguousarray(back(out)), ref["retrace"])
    out = B.rlcs_td_lambda_time_major(r, v, d, tr, bv, bt, gamma=p["gamma"], lam=p["lam"])
    assert_close("td_lambda", np.ascontiguousarray(back(out)), ref["td_lambda"])
    out = B.rlcs_discounted_return_time_major(r, d, tr, bv, bt, gamma=p["gamma"])
    assert_close("disc", np.ascontiguousarray(back(out)), ref["discounted_return"])
    out = B.rlcs_elig_trace_time_major(x, dany, gamma=p["gamma"], lam=p["lam"])
    assert_close("elig", np.ascontiguousarray(back(out)), ref["elig_trace"])
    out = B.rlcs_episodic_prefix_sum_time_major(x, dany)
    assert_close("prefix ends_at", np.ascontiguousarray(back(out)), ref["prefix_ends_at"])
    out = B.rlcs_episodic_prefix_sum_time_major(x, dany, starts_at=True)
    assert_close("prefix starts_at", np.ascontiguousarray(back(out)), ref["prefix_starts_at"])
    # NULL truncs / bootstrap
    ref2 = run_oracle(oracle, ro, ("gae", "discounted_return"), use_truncs=False, use_bootstrap=False)
    adv2 = B.rlcs_gae_time_major(r, v, d, gamma=p["gamma"], lam=p["lam"], want_returns=False)
    assert_close("gae no truncs", np.ascontiguousarray(back(adv2)), ref2["gae"][0])
    adv3, ret3 = B.rlcs_gae_time_major(r, v, d, gamma=p["gamma"], lam=p["lam"])
    assert_close("gae no truncs, with returns", np.ascontiguousarray(back(ret3)), ref2["gae"][1])
    ref3 = run_oracle(oracle, ro, ("td_lambda",), use_truncs=False)
    out = B.rlcs_td_lambda_time_major(r, v, d, None, None, bt, gamma=p["gamma"], lam=p["lam"])
    assert_close("td_lambda no truncs", np.ascontiguousarray(back(out)), ref3["td_lambda"])
    out = B.rlcs_discounted_return_time_major(r, d, gamma=p["gamma"])
    assert_close("disc no truncs", np.ascontiguousarray(back(out)), ref2["discounted_return"])


def test_time_major_paths_agree_and_misaligned_inputs_fall_back(oracle, W, B):
    """Block kernel (shared-memory ring, time split among warps) and register walk agree to rounding;
    inputs that are only 4-byte aligned take the register walk silently, with identical bits."""
    import torch
    N, T = 4112, 300
    ro = W.make_rollout(116, N, T, p_done=0.03, p_trunc=0.01)
    p = ro.params
    names = ("rewards", "values", "dones", "truncs", "trunc_bootstrap")
    al = [_tm(getattr(ro, k)) for k in names]
    bt = guarded_upload(ro.bootstrap)
    outs = []
    for path in (1, 2):
        B.rlcs_debug_time_major_path(path)
        try:
            outs.append(B.rlcs_gae_time_major(*al, bt, gamma=p["gamma"], lam=p["lam"]))
        finally:
            B.rlcs_debug_time_major_path(0)
    assert_close("adv ring vs walk", outs[1][0].cpu().numpy(), outs[0][0].cpu().numpy().astype(np.float64))
    assert_close("ret ring vs walk", outs[1][1].cpu().numpy(), outs[0][1].cpu().numpy().astype(np.float64))
    # the same tensors one element into a larger allocation: 4-byte (1-byte for masks) aligned only
    mis = []
    for a in al:
        mis.append(guarded_upload(a.cpu(), 1))
    out = B.rlcs_gae_time_major(*mis, bt, gamma=p["gamma"], lam=p["lam"])
    assert torch.equal(out[0], outs[0][0]) and torch.equal(out[1], outs[0][1])


@pytest.mark.parametrize("N,T,p_flag", [(64, 3000, 0.0), (64, 3000, 0.01), (16, 20000, 0.0005), (2048, 700, 0.0)])
def test_time_major_chained_kernel_is_reproducible_and_agrees_with_three_launches(oracle, W, B, N, T, p_flag):
    """Cut time axis: the single chained launch gives the same bits run after run (its look-back
    re-applies aggregates in a fixed order whatever the timing), and agrees to rounding with the
    three-launch path.  Without flags every carry chain runs the whole window."""
    import torch
    ro = W.make_rollout(118, N, T, p_done=p_flag, p_trunc=p_flag / 2)
    p = ro.params
    al = [_tm(getattr(ro, k)) for k in ("rewards", "values", "dones", "truncs", "trunc_bootstrap")]
    bt = guarded_upload(ro.bootstrap)
    x, dany = _tm(ro.x), _tm(ro.any_done)
    outs = {}
    for path in (5, 5, 4):
        B.rlcs_debug_time_major_path(path)
        try:
            need = int(B.lib().rlcs_time_major_workspace_bytes(N, T))
            ws = B.Workspace(N, T, nbytes=need)
            adv, ret = B.rlcs_gae_time_major(*al, bt, gamma=p["gamma"], lam=p["lam"], workspace=ws)
            z = B.rlcs_elig_trace_time_major(x, dany, gamma=p["gamma"], lam=p["lam"], workspace=ws)
            torch.cuda.synchronize()
            assert ws.device_status() == B.RLCS_OK
            outs.setdefault(path, []).append((adv, ret, z))
        finally:
            B.rlcs_debug_time_major_path(0)
    for a, b in zip(outs[5][0], outs[5][1]):
        assert torch.equal(a, b)
    for a, b in zip(outs[5][0], outs[4][0]):
        assert_close("chained vs three launches", a.cpu().numpy(), b.cpu().numpy().astype(np.float64))
    ref = run_oracle(oracle, ro, ("gae", "elig_trace"))
    assert_close("chained gae", np.ascontiguousarray(outs[5][0][0].cpu().numpy().T), ref["gae"][0])
    assert_close("chained elig", np.ascontiguousarray(outs[5][0][2].cpu().numpy().T), ref["elig_trace"])


def test_time_major_chained_wait_runs_out_and_reports_timeout(oracle, W, B):
    """A block that never publishes its chunk: the waits of the chunks after it run out of polls,
    the kernel finishes, the status word says TIMEOUT, and the next call on the workspace is right."""
    import torch
    N, T = 64, 4096
    ro = W.make_rollout(119, N, T, p_done=0.0, p_trunc=0.0)
    p = ro.params
    r, d = _tm(ro.rewards), _tm(ro.dones)
    ws = B.Workspace(N, T, nbytes=int(B.lib().rlcs_time_major_workspace_bytes(N, T)))
    B.rlcs_debug_set_carry_fault(2, 50)
    try:
        B.rlcs_discounted_return_time_major(r, d, gamma=p["gamma"], workspace=ws)
        torch.cuda.synchronize()
        assert ws.device_status() == B.RLCS_ERR_TIMEOUT
    finally:
        B.rlcs_debug_set_carry_fault(-1, 0)
    assert ws.device_status() == B.RLCS_OK
    out = B.rlcs_discounted_return_time_major(r, d, gamma=p["gamma"], workspace=ws)
    ref = run_oracle(oracle, ro, ("discounted_return",), use_truncs=False, use_bootstrap=False)
    assert_close("after the timeout", np.ascontiguousarray(out.cpu().numpy().T), ref["discounted_return"])
    assert ws.device_status() == B.RLCS_OK


def test_time_major_argument_checks(oracle, W, B):
    L = B.lib()
    P = 0x7f0000000000
    g = lambda **k: L.rlcs_gae_time_major(k.get("r", P), P, k.get("d", P), k.get("tr"), k.get("bv"), None, P, None,
                                          k.get("N", 4), k.get("T", 8), k.get("g", 0.9), 0.9, None, 0, None)
    assert g(N=0) == B.RLCS_OK and g(N=-1) == B.RLCS_ERR_SIZE and g(g=2.0) == B.RLCS_ERR_ARG
    assert g(r=None) == B.RLCS_ERR_NULL and g(d=None) == B.RLCS_ERR_NULL and g(tr=P) == B.RLCS_ERR_NULL
    assert g(r=P + 2) == B.RLCS_ERR_ALIGN
    assert L.rlcs_time_major_workspace_bytes(100000, 64) == 0 and L.rlcs_time_major_workspace_bytes(8, 4096) > 0
    assert g(N=8, T=4096) == B.RLCS_ERR_WORKSPACE


def test_randomized_time_major_and_skip(oracle, W, B):
    """Seeded fuzz of the entry points beyond the paper's API: time-major (both kernels, every warp
    count and chunking the planner picks), GAE with observation-skip masking."""
    import torch
    rng = np.random.default_rng(20260818)
    for case in range(40):
        N = int(rng.choice([rng.integers(1, 64), 16 * rng.integers(1, 40), 16 * rng.integers(200, 1300)]))
        T = int(rng.choice([rng.integers(1, 40), rng.integers(40, 700), rng.integers(700, 5000)]))
        if N * T > 1_500_000:
            T = max(1, 1_500_000 // N)
        p_done = float(rng.choice([0.0, 0.01, 0.3]))
        ro = W.make_rollout(131, N, T, p_done=p_done, p_trunc=float(rng.choice([0.0, 0.01, 0.2])), salt=case)
        ro.params.update(gamma=float(rng.choice([0.9, 0.99, 1.0])), lam=float(rng.choice([0.0, 0.5, 0.95, 1.0])))
        p = ro.params
        use_tr, use_bt = bool(rng.random() < 0.7), bool(rng.random() < 0.8)
        ref = run_oracle(oracle, ro, ALL_ALGOS, use_truncs=use_tr, use_bootstrap=use_bt)
        tm = lambda a: None if a is None else _tm(a)
        r, v, d, q, eq, lr, x, dany = (tm(getattr(ro, k)) for k in ("rewards", "values", "dones", "q_sa", "expected_q", "log_rhos", "x", "any_done"))
        tr, bv = (tm(ro.truncs), tm(ro.trunc_bootstrap)) if use_tr else (None, None)
        bt = guarded_upload(ro.bootstrap) if use_bt else None
        back = lambda t: np.ascontiguousarray(t.cpu().numpy().T)
        path = int(rng.choice([0, 1, 3]))
        B.rlcs_debug_time_major_path(path)
        try:
            adv, ret = B.rlcs_gae_time_major(r, v, d, tr, bv, bt, gamma=p["gamma"], lam=p["lam"])
            vs, pg = B.rlcs_vtrace_time_major(r, v, lr, d, tr, bv, bt, gamma=p["gamma"], rho_bar=p["rho_bar"], c_bar=p["c_bar"])
            qt = B.rlcs_retrace_time_major(r, q, eq, lr, d, tr, bv, bt, gamma=p["gamma"], lam=p["lam"], c_bar=p["c_bar"])
            td = B.rlcs_td_lambda_time_major(r, v, d, tr, bv, bt, gamma=p["gamma"], lam=p["lam"])
            dr = B.rlcs_discounted_return_time_major(r, d, tr, bv, bt, gamma=p["gamma"])
            el = B.rlcs_elig_trace_time_major(x, dany, gamma=p["gamma"], lam=p["lam"])
            ps = B.rlcs_episodic_prefix_sum_time_major(x, dany, starts_at=bool(case % 2))
        finally:
            B.rlcs_debug_time_major_path(0)
        tag = f"case {case}: N={N} T={T} path={path} truncs={use_tr} boot={use_bt}"
        for name, got, want in (("gae", adv, ref["gae"][0]), ("ret", ret, ref["gae"][1]), ("vs", vs, ref["vtrace"][0]),
                                ("pg", pg, ref["vtrace"][1]), ("retrace", qt, ref["retrace"]), ("td", td, ref["td_lambda"]),
                                ("disc", dr, ref["discounted_return"]), ("elig", el, ref["elig_trace"]),
                                ("prefix", ps, ref["prefix_starts_at" if case % 2 else "prefix_ends_at"])):
            assert_close(f"{tag} {name}", back(got), want)
        # observation-skip masking on the same rollout (row-major)
        skip = (rng.random((N, T)) < float(rng.choice([0.0, 0.3, 0.8]))).astype(np.uint8)
        dev = Dev(ro, offset=int(rng.choice([0, 0, 1])))
        sk = guarded_upload(skip, dev.offset)
        a, rt, fil = B.rlcs_gae_skip(dev.rewards, dev.values, dev.dones, dev.truncs if use_tr else None,
                                     dev.trunc_bootstrap if use_tr else None, dev.bootstrap if use_bt else None, skip=sk,
                                     gamma=p["gamma"], lam=p["lam"], values_filled=dev.empty_out(), advantages=dev.empty_out(),
                                     returns=dev.empty_out(), workspace=B.Workspace(N, T))
        ra, rr, rf = oracle.gae_skip(ro.rewards, ro.values, ro.dones, ro.truncs if use_tr else None,
                                     ro.trunc_bootstrap if use_tr else None, ro.bootstrap if use_bt else None, skip=skip,
                                     gamma=p["gamma"], lam=p["lam"])
        assert_close(f"{tag} skip adv", a.cpu().numpy(), ra)
        assert_close(f"{tag} skip ret", rt.cpu().numpy(), rr)
        assert np.array_equal(fil.cpu().numpy().astype(np.float64), rf), tag


def test_calls_can_be_captured_in_a_cuda_graph(oracle, W, B):
    """No entry point allocates, synchronises or keeps host state a replay would miss: a graph that
    captured one call of each family reproduces the eager results bit for bit, twice (the second
    replay also proves that the carry workspace's per-call epoch advances inside the graph)."""
    import torch
    ro = W.make_rollout(132, 48, 3000, p_done=0.01, p_trunc=0.01)         # rows straddle tiles: look-back runs
    p = ro.params
    dev = Dev(ro)
    r_tm, v_tm, d_tm = _tm(ro.rewards), _tm(ro.values), _tm(ro.dones)
    tr_tm, bv_tm = _tm(ro.truncs), _tm(ro.trunc_bootstrap)
    skip = (torch.rand((ro.N, ro.T), device="cuda") < 0.3).to(torch.uint8)
    r16, v16 = dev.rewards.to(torch.bfloat16), dev.values.to(torch.bfloat16)
    bv16, bt16 = dev.trunc_bootstrap.to(torch.bfloat16), dev.bootstrap.to(torch.bfloat16)
    ws = B.Workspace(ro.N, ro.T)
    wsn = B.Workspace(ro.N, ro.T, nbytes=int(B.lib().rlcs_gae_normalized_workspace_bytes(ro.N, ro.T)))
    wtm = B.Workspace(ro.N, ro.T, nbytes=max(256, int(B.lib().rlcs_time_major_workspace_bytes(ro.N, ro.T))))
    new = lambda like=dev.rewards, dt=None: guarded_empty(tuple(like.shape), dt or like.dtype)
    outs = {k: new() for k in ("adv", "ret", "vs", "pg", "q", "nadv", "nret", "sadv", "sret", "fil", "el")}
    outs.update(tadv=new(r_tm), tret=new(r_tm), badv=new(dt=torch.bfloat16), bret=new(dt=torch.bfloat16))

    def run(s):
        kw = dict(stream=s)
        B.rlcs_gae(dev.rewards, dev.values, dev.dones, dev.truncs, dev.trunc_bootstrap, dev.bootstrap, gamma=p["gamma"],
                   lam=p["lam"], advantages=outs["adv"], returns=outs["ret"], workspace=ws, **kw)
        B.rlcs_vtrace(dev.rewards, dev.values, dev.log_rhos, dev.dones, dev.truncs, dev.trunc_bootstrap, dev.bootstrap,
                      gamma=p["gamma"], vs=outs["vs"], pg_advantages=outs["pg"], workspace=ws, **kw)
        B.rlcs_retrace(dev.rewards, dev.q_sa, dev.expected_q, dev.log_rhos, dev.dones, dev.truncs, dev.trunc_bootstrap,
                       dev.bootstrap, gamma=p["gamma"], lam=p["lam"], q_targets=outs["q"], workspace=ws, **kw)
        B.rlcs_elig_trace(dev.x, dev.any_done, gamma=p["gamma"], lam=p["lam"], traces=outs["el"], workspace=ws, **kw)
        B.rlcs_gae_normalized(dev.rewards, dev.values, dev.dones, dev.truncs, dev.trunc_bootstrap, dev.bootstrap,
                              gamma=p["gamma"], lam=p["lam"], advantages=outs["nadv"], returns=outs["nret"], workspace=wsn, **kw)
        B.rlcs_gae_skip(dev.rewards, dev.values, dev.dones, dev.truncs, dev.trunc_bootstrap, dev.bootstrap, skip=skip,
                        gamma=p["gamma"], lam=p["lam"], values_filled=outs["fil"], advantages=outs["sadv"],
                        returns=outs["sret"], workspace=ws, **kw)
        B.rlcs_gae_time_major(r_tm, v_tm, d_tm, tr_tm, bv_tm, dev.bootstrap, gamma=p["gamma"], lam=p["lam"],
                              advantages=outs["tadv"], returns=outs["tret"], workspace=wtm, **kw)
        B.rlcs_gae_bf16(r16, v16, dev.dones, dev.truncs, bv16, bt16, gamma=p["gamma"], lam=p["lam"],
                        advantages=outs["badv"], returns=outs["bret"], workspace=ws, **kw)

    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        run(s)                                                   # eager (also the warm-up before capture)
        torch.cuda.synchronize()
        eager = {k: v.clone() for k, v in outs.items()}
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=s):
            run(s)
        for _ in range(2):
            for v in outs.values():
                v.zero_()
            graph.replay()
            torch.cuda.synchronize()
            for k, v in outs.items():
                assert torch.equal(v.view(torch.int16 if v.dtype == torch.bfloat16 else torch.int32),
                                   eager[k].view(torch.int16 if v.dtype == torch.bfloat16 else torch.int32)), k
    assert ws.device_status() == 0 and wsn.device_status() == 0
    assert_close("graph gae", outs["adv"].cpu().numpy(), run_oracle(oracle, ro, ("gae",))["gae"][0])


# ------------------------------------------------------------------ test hooks
def test_affine_scan_matches_generic_recurrence(oracle, W, B):
    import torch
    rng = np.random.default_rng(5)
    N, T = 4, 3000
    alpha = rng.standard_normal((N, T)).astype(np.float32)
    beta = rng.uniform(0.0, 1.0, (N, T)).astype(np.float32)
    beta[rng.random((N, T)) < 0.01] = 0.0
    ws = B.Workspace(N, T)
    for fwd in (False, True):
        out = B.rlcs_affine_scan(guarded_upload(alpha), guarded_upload(beta), forward=fwd,
                                 workspace=ws).cpu().numpy()
        ref = np.stack([oracle.linear_recurrence(alpha[n].astype(np.float64), beta[n].astype(np.float64), 0.0,
                                                 forward=fwd) for n in range(N)])
        assert_close(f"affine fwd={fwd}", out, ref)


def test_bounded_carry_wait_reports_timeout_and_returns(oracle, W, B):
    """A tile that never publishes: its dependant's wait runs out of polls, the kernel finishes,
    the status word says TIMEOUT, and the next call on the same workspace works again."""
    import torch
    ro = W.make_rollout(104, 1, 16384, p_done=0.0, p_trunc=0.0)
    dev = Dev(ro)
    ws = B.Workspace(ro.N, ro.T)
    B.rlcs_debug_set_carry_fault(2, 64)
    B.rlcs_debug_allow_cluster_carry(False)           # this row length would otherwise carry on chip
    try:
        B.rlcs_discounted_return(dev.rewards, dev.dones, gamma=0.99, workspace=ws)
        torch.cuda.synchronize()
        assert ws.device_status() == B.RLCS_ERR_TIMEOUT
    finally:
        B.rlcs_debug_set_carry_fault(-1, 0)
        B.rlcs_debug_allow_cluster_carry(True)
    assert ws.device_status() == B.RLCS_OK            # cleared by the read
    compare_all(oracle, ro, algos=("discounted_return",), workspace=ws)


def test_missing_workspace_is_an_error_not_a_launch(oracle, W, B):
    ro = W.make_rollout(105, 2, 3000)
    dev = Dev(ro)
    with pytest.raises(B.RlcsError) as e:
        B.rlcs_discounted_return(dev.rewards, dev.dones, gamma=0.99, workspace=None)
    assert e.value.status == B.RLCS_ERR_WORKSPACE
    small = B.Workspace(2, 3000, nbytes=256)
    with pytest.raises(B.RlcsError) as e:
        B.rlcs_discounted_return(dev.rewards, dev.dones, gamma=0.99, workspace=small)
    assert e.value.status == B.RLCS_ERR_WORKSPACE
