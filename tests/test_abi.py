"""Host-side checks that need no GPU: the library builds and loads, exports every symbol the
header declares, and rejects bad arguments before anything is launched (no compute calls here)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

OK, E_NULL, E_SIZE, E_ARG, E_ALIGN, E_WS = 0, 1, 2, 3, 4, 5


@pytest.fixture(scope="module")
def L():
    from paper_2608_17641_b200 import build, binding
    build.build()
    return binding.lib()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "rlcs.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(rlcs_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_seven_entry_points():
    names = _declared_symbols()
    for n in ("rlcs_gae", "rlcs_vtrace", "rlcs_retrace", "rlcs_td_lambda", "rlcs_discounted_return",
              "rlcs_elig_trace", "rlcs_episodic_prefix_sum", "rlcs_workspace_bytes", "rlcs_workspace_init",
              "rlcs_last_device_status", "rlcs_status_string"):
        assert n in names


def test_library_exports_every_declared_symbol(L):
    from paper_2608_17641_b200 import binding
    for name in _declared_symbols():
        assert hasattr(L, name), f"{name} declared in rlcs.h but not exported"
        assert name in binding.SIGNATURES, f"{name} has no binding signature"
    for name in binding.SIGNATURES:
        assert name in _declared_symbols(), f"binding knows {name} but rlcs.h does not declare it"


def test_no_alloc_limit_is_decided_on_the_scratch_a_call_uses(L):
    cap = L.rlcs_no_alloc_scratch_bytes()
    assert cap == 1 << 20
    assert L.rlcs_gae_carry_bytes(0, 5, 0, 1) == 0 and L.rlcs_gae_carry_bytes(-1, 5, 0, 1) == 0
    for N, T in ((96, 999), (8, 128), (4096, 999), (33545, 999)):
        for tr in (0, 1):
            for vec in (0, 1):
                assert L.rlcs_gae_carry_bytes(N, T, tr, vec) <= L.rlcs_workspace_bytes(N, T)
    assert L.rlcs_gae_carry_bytes(16384, 2048, 1, 1) == 0 and L.rlcs_gae_carry_bytes(64, 16384, 0, 1) == 0
    assert L.rlcs_gae_carry_bytes(33545, 999, 1, 1) <= cap < L.rlcs_gae_carry_bytes(140000, 999, 0, 1)
    # beyond the array: refused on the host, before anything touches a device
    assert L.rlcs_gae_no_alloc(P, P, P, None, None, None, P, None, 140000, 999, 0.99, 0.95, None) == 8
    assert b"scratch" in L.rlcs_status_string(8) and b"capture" in L.rlcs_status_string(9)


def test_row_aligned_tiling_needs_no_carry_workspace(L):
    """Short rows that nearly fill a tile with a whole number of rows are tiled by rows: no carry."""
    try:
        for N, T in ((4096, 1000), (16384, 2000), (4096, 500), (4096, 250), (64, 200)):
            assert L.rlcs_gae_carry_bytes(N, T, 1, 1) == 0, (N, T)
        assert L.rlcs_gae_carry_bytes(4096, 999, 1, 1) > 0          # 999 steps do not split into whole chunks
        assert L.rlcs_gae_carry_bytes(4096, 600, 1, 1) > 0          # one row would leave 41 % of the tile idle
        assert L.rlcs_gae_carry_bytes(64, 3000, 1, 1) > 0           # rows longer than a tile
        assert L.rlcs_debug_allow_row_tiles(0) == OK
        assert L.rlcs_gae_carry_bytes(4096, 1000, 1, 1) > 0
    finally:
        L.rlcs_debug_allow_row_tiles(1)


def test_one_block_per_row_needs_no_carry_workspace_except_for_a_thin_second_wave(L):
    """Long rows of whole tiles, enough of them: one thread block per row, no carry workspace -- unless the
    rows are a little more than the blocks the GPU holds at once (148 SMs x 6 blocks here: 888), where the
    few blocks of the second wave would finish the call alone and the carry between blocks is kept."""
    T = 32768                                                       # 16 tiles of 2048: too long for a cluster per row
    assert L.rlcs_gae_carry_bytes(800, T, 1, 1) == 0
    assert L.rlcs_gae_carry_bytes(888, T, 1, 1) == 0
    assert L.rlcs_gae_carry_bytes(900, T, 1, 1) > 0
    assert L.rlcs_gae_carry_bytes(1060, T, 1, 1) > 0
    assert L.rlcs_gae_carry_bytes(1100, T, 1, 1) == 0
    assert L.rlcs_gae_carry_bytes(300, T, 1, 1) > 0                 # fewer than three rows per SM
    try:
        assert L.rlcs_debug_set_row_blocks(1) == OK                 # forced: any number of rows
        assert L.rlcs_gae_carry_bytes(900, T, 1, 1) == 0 and L.rlcs_gae_carry_bytes(3, T, 1, 1) == 0
        assert L.rlcs_debug_set_row_blocks(0) == OK                 # never
        assert L.rlcs_gae_carry_bytes(800, T, 1, 1) > 0
    finally:
        L.rlcs_debug_set_row_blocks(-1)


def test_status_strings(L):
    assert L.rlcs_status_string(0) == b"RLCS_OK"
    for s in range(1, 8):
        assert L.rlcs_status_string(s).startswith(b"RLCS_ERR_")
    assert b"unknown" in L.rlcs_status_string(99)


def test_workspace_bytes(L):
    assert L.rlcs_workspace_bytes(0, 128) == 0 and L.rlcs_workspace_bytes(8, 0) == 0
    assert L.rlcs_workspace_bytes(-1, 5) == 0
    for T in (1, 2, 64, 128, 512):                      # T divides every tile: nothing straddles
        assert L.rlcs_workspace_bytes(4096, T) == 0
    assert L.rlcs_workspace_bytes(64, 16384) == 256 + 16 * (64 * 16384 // 512 + 1)
    assert L.rlcs_workspace_bytes(3, 1000) == 256 + 16 * ((3000 + 511) // 512 + 1)


# fake, never-dereferenced device addresses: every call below must return before any launch
P = 0x7f0000000000
Q = P + 4                                                # 4-byte but not 16-byte aligned
ODD = P + 2                                              # not even 4-byte aligned


def _gae(L, r=P, v=P, d=P, tr=None, bv=None, bt=None, adv=P, ret=None, N=4, T=8, g=0.99, l=0.95, ws=None, wsb=0):
    return L.rlcs_gae(r, v, d, tr, bv, bt, adv, ret, N, T, g, l, ws, wsb, None)


def test_empty_problem_is_ok_without_launch(L):
    assert _gae(L, N=0) == OK and _gae(L, T=0) == OK
    assert L.rlcs_elig_trace(None, None, None, 0, 5, 0.9, 0.9, None, 0, None) == OK


def test_size_errors(L):
    assert _gae(L, N=-1) == E_SIZE and _gae(L, T=-3) == E_SIZE
    assert _gae(L, T=2 ** 31) == E_SIZE
    assert _gae(L, N=2 ** 40, T=2 ** 20) == E_SIZE


def test_parameter_errors(L):
    for g, l in [(-0.1, 0.5), (1.1, 0.5), (0.5, -1e-3), (0.5, 1.5), (float("nan"), 0.5), (0.5, float("nan"))]:
        assert _gae(L, g=g, l=l) == E_ARG
    v = lambda rb, cb: L.rlcs_vtrace(P, P, P, P, None, None, None, P, None, 4, 8, 0.9, rb, cb, None, 0, None)
    assert v(-1.0, 1.0) == E_ARG and v(1.0, float("nan")) == E_ARG
    assert L.rlcs_retrace(P, P, P, P, P, None, None, None, P, 4, 8, 0.9, 2.0, 1.0, None, 0, None) == E_ARG
    assert L.rlcs_discounted_return(P, P, None, None, None, P, 4, 8, 7.0, None, 0, None) == E_ARG
    assert L.rlcs_elig_trace(P, P, P, 4, 8, 0.9, -0.5, None, 0, None) == E_ARG


def test_null_pointer_errors(L):
    assert _gae(L, r=None) == E_NULL and _gae(L, v=None) == E_NULL
    assert _gae(L, d=None) == E_NULL and _gae(L, adv=None) == E_NULL
    assert _gae(L, tr=P, bv=None) == E_NULL and _gae(L, tr=None, bv=P) == E_NULL
    assert L.rlcs_episodic_prefix_sum(P, None, P, 4, 8, 0, None, 0, None) == E_NULL
    assert L.rlcs_affine_scan(P, None, P, 4, 8, 0, None, 0, None) == E_NULL


def test_retrace_probs_argument_checks(L):
    f = lambda **k: L.rlcs_retrace_probs(k.get("r", P), k.get("q", P), k.get("pi", P), k.get("mu", P), k.get("act", P), P,
                                         None, None, None, P, k.get("N", 4), k.get("T", 8), k.get("A", 4), k.get("g", 0.9),
                                         0.9, k.get("c", 1.0), None, 0, None)
    assert f(A=0) == E_SIZE and f(A=2 ** 21) == E_SIZE and f(N=2 ** 30, T=2 ** 9, A=2 ** 10) == E_SIZE
    assert f(g=1.5) == E_ARG and f(c=-1.0) == E_ARG
    assert f(q=None) == E_NULL and f(pi=None) == E_NULL and f(mu=None) == E_NULL and f(act=None) == E_NULL
    assert f(q=ODD) == E_ALIGN and f(act=ODD) == E_ALIGN
    assert f(N=0) == OK


def test_alignment_errors(L):
    assert _gae(L, r=ODD) == E_ALIGN
    assert _gae(L, adv=ODD) == E_ALIGN
    # rows straddle tiles at T = 1000: a workspace is required, 16-byte aligned, large enough
    need = L.rlcs_workspace_bytes(4, 1000)
    assert need > 0
    assert _gae(L, N=4, T=1000) == E_WS
    assert _gae(L, N=4, T=1000, ws=P, wsb=need - 16 * 8) == E_WS
    assert _gae(L, N=4, T=1000, ws=Q, wsb=need) == E_ALIGN


def test_workspace_init_argument_checks(L):
    assert L.rlcs_workspace_init(None, 0, None) == OK
    assert L.rlcs_workspace_init(None, 64, None) == E_NULL
    assert L.rlcs_workspace_init(Q, 4096, None) == E_ALIGN
    assert L.rlcs_workspace_init(P, 8, None) == E_WS
    assert L.rlcs_last_device_status(None, None) == OK


def test_debug_hooks_argument_checks(L):
    assert L.rlcs_debug_set_tile_variant(99) == E_ARG and L.rlcs_debug_set_tile_variant(-2) == E_ARG
    assert L.rlcs_debug_set_tile_variant(-1) == OK
    assert L.rlcs_debug_set_tile_variant(0) == OK
    assert L.rlcs_debug_tile_elems(0) == 2048 and L.rlcs_debug_tile_elems(1) == 512
    assert L.rlcs_debug_tile_elems(99) == 0


def test_binding_rejects_cpu_tensors_and_wrong_dtypes():
    import torch
    from paper_2608_17641_b200 import binding
    x = torch.zeros(2, 8)
    d = torch.zeros(2, 8, dtype=torch.uint8)
    with pytest.raises(TypeError):                       # no CPU path: CUDA tensors only
        binding.rlcs_elig_trace(x, d, gamma=0.9, lam=0.9, traces=x.clone())


class _FakeDevice:
    def __init__(self, index):
        self.index = index


class _FakeTensor:
    """Stands in for a CUDA tensor on a chosen device (no GPU is needed to check the host-side rule)."""

    def __init__(self, index, dtype=None, shape=(2, 8)):
        import torch
        self.is_cuda, self.device, self.dtype, self.shape = True, _FakeDevice(index), dtype or torch.float32, shape

    def is_contiguous(self):
        return True

    def get_device(self):
        return self.device.index

    def data_ptr(self):
        return 0x7f0000000000 + 4096 * (self.device.index or 0)


def test_binding_rejects_tensors_and_workspaces_of_another_device(monkeypatch):
    """The library launches on the current device: a tensor or workspace of another GPU is refused
    on the host instead of reaching a kernel as a foreign pointer."""
    from paper_2608_17641_b200 import binding
    monkeypatch.setattr(binding, "_current_device", lambda: 0)
    assert binding._ptr(_FakeTensor(0), "f32", (2, 8)) == 0x7f0000000000
    with pytest.raises(ValueError, match="cuda:1 but the current device is cuda:0"):
        binding._ptr(_FakeTensor(1), "f32", (2, 8))
    ws = binding.Workspace.__new__(binding.Workspace)
    ws.nbytes, ws.buf = 1024, _FakeTensor(1)
    with pytest.raises(ValueError, match="workspace is on cuda:1"):
        binding._ws(ws)
    ws.buf = _FakeTensor(0)
    assert binding._ws(ws) == (ws.buf.data_ptr(), 1024)
    monkeypatch.setattr(binding, "_current_device", lambda: 1)
    with pytest.raises(ValueError):
        binding._ptr(_FakeTensor(0), "f32")


def test_prepare_records_the_call_instead_of_making_it(monkeypatch):
    """prepare() runs a wrapper with all its checks but makes no launch: it returns the C function and
    the marshalled arguments, to be repeated at C-call cost."""
    import torch
    from paper_2608_17641_b200 import binding
    binding.lib()
    monkeypatch.setattr(binding, "_current_device", lambda: 0)
    monkeypatch.setattr(binding, "_stream", lambda stream=None: 1234)
    x, d, z = _FakeTensor(0), _FakeTensor(0, torch.uint8), _FakeTensor(0)
    step = binding.prepare(binding.rlcs_elig_trace, x, d, gamma=0.9, lam=0.5, traces=z)
    assert step.outputs is z and len(step._calls) == 1
    fn, args = step._calls[0]
    assert fn is binding.lib().rlcs_elig_trace                     # the library is back in place
    assert args[0] == x.data_ptr() and args[2] == z.data_ptr() and tuple(args[3:5]) == (2, 8) and args[-1] == 1234
    with pytest.raises(TypeError):                                   # checks still run at prepare time
        binding.prepare(binding.rlcs_elig_trace, _FakeTensor(0, torch.float64), d, gamma=0.9, lam=0.5, traces=z)
    assert not isinstance(binding.lib(), binding._Recorder)
    with pytest.raises(ValueError):
        binding.prepare(lambda: None)


def test_front_end_keeps_one_workspace_per_stream(monkeypatch):
    """Calls on different streams must not share carry records: the cache key holds the stream."""
    from paper_2608_17641_b200 import api

    class FakeStream:
        def __init__(self, handle):
            self.cuda_stream = handle

    made = []

    class FakeWorkspace:
        def __init__(self, N, T, device=None, stream=None, nbytes=None):
            made.append((N, T, stream.cuda_stream, nbytes))

    monkeypatch.setattr(api._B, "Workspace", FakeWorkspace)
    monkeypatch.setattr(api, "_workspaces", {})
    like = _FakeTensor(0)
    a = api._workspace(like, 4, 1000, stream=FakeStream(11))
    b = api._workspace(like, 4, 1000, stream=FakeStream(11))
    c = api._workspace(like, 4, 1000, stream=FakeStream(22))
    assert a is b and a is not c and [m[2] for m in made] == [11, 22]


def test_missing_library_fails_loudly(tmp_path, monkeypatch):
    from paper_2608_17641_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no fallback"):
        binding.lib()


# ------------------------------------------------------------------ the entry points beyond the paper's API
def test_time_major_validation_and_workspace_plan(L):
    tm = lambda **k: L.rlcs_gae_time_major(k.get("r", P), P, k.get("d", P), k.get("tr"), k.get("bv"), None, P, None,
                                           k.get("N", 4), k.get("T", 8), k.get("g", 0.9), 0.9, None, 0, None)
    assert tm(N=0) == OK and tm(N=-1) == E_SIZE and tm(T=2 ** 31) == E_SIZE and tm(g=2.0) == E_ARG
    assert tm(r=None) == E_NULL and tm(d=None) == E_NULL and tm(tr=P) == E_NULL and tm(r=ODD) == E_ALIGN
    # enough environments: whole columns, no workspace; few environments: the time axis is cut
    assert L.rlcs_time_major_workspace_bytes(100000, 64) == 0 and L.rlcs_time_major_workspace_bytes(3072, 5000) == 0
    need = L.rlcs_time_major_workspace_bytes(8, 4096)
    # header, then the larger of: one 16-byte record per 64-step chunk and (padded) column, two floats per chunk and column
    assert need == 256 + 16 * 64 * (4096 // 64)
    assert L.rlcs_time_major_workspace_bytes(8, 40) == 0   # chunks are at least 64 steps
    assert tm(N=8, T=4096) == E_WS
    assert L.rlcs_elig_trace_time_major(None, P, P, 4, 8, 0.9, 0.9, None, 0, None) == E_NULL
    assert L.rlcs_episodic_prefix_sum_time_major(P, P, P, 0, 8, 0, None, 0, None) == OK


def test_bf16_validation(L):
    g = lambda **k: L.rlcs_gae_bf16(k.get("r", P), P, P, k.get("tr"), None, None, P, None, k.get("N", 4), k.get("T", 128),
                                    k.get("g", 0.9), 0.9, None, 0, None)
    assert g(N=0) == OK and g(N=-1) == E_SIZE and g(g=-0.1) == E_ARG and g(r=None) == E_NULL and g(tr=P) == E_NULL
    assert g(r=P + 1) == E_ALIGN and g(N=3, T=3000) == E_WS
    assert L.rlcs_retrace_bf16(P, P, None, P, P, None, None, None, P, 4, 128, 0.9, 0.9, 1.0, None, 0, None) == E_NULL
    assert L.rlcs_vtrace_bf16(P, P, P, P, None, None, None, P, None, 4, 128, 0.9, -1.0, 1.0, None, 0, None) == E_ARG


def test_vector_trace_and_skip_validation(L):
    assert L.rlcs_elig_trace_vec_beta(P, P, P, P, 4, 8, 0, None, 0, None) == OK
    assert L.rlcs_elig_trace_vec_beta(P, None, P, P, 4, 8, 4, None, 0, None) == E_NULL
    assert L.rlcs_elig_trace_vec_beta(P, ODD, P, P, 4, 8, 4, None, 0, None) == E_ALIGN
    assert L.rlcs_elig_trace_vec_beta_workspace_bytes(2, 100000, 8) > L.rlcs_elig_trace_vec_workspace_bytes(2, 100000, 8) > 0
    assert L.rlcs_elig_trace_vec_beta(P, P, P, P, 2, 100000, 8, None, 0, None) == E_WS
    sk = lambda **k: L.rlcs_gae_skip(P, P, P, None, None, None, k.get("sk", P), k.get("fil", P), P, None, k.get("N", 4), 128,
                                     k.get("g", 0.9), 0.9, None, 0, None)
    assert sk(N=0) == OK and sk(sk=None) == E_NULL and sk(fil=None) == E_NULL and sk(g=1.5) == E_ARG and sk(fil=ODD) == E_ALIGN
