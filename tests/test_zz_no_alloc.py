"""rlcs_gae_no_alloc: the GAE entry point for callers that cannot allocate device memory (its carry
scratch is a fixed array inside the library).  Called through the C ABI twice in a row and compared
with rlcs_gae on a caller-provided workspace; kept in a file of its own that pytest collects last."""
import numpy as np
import pytest

from _util import ATOL, RTOL, Dev, assert_close

pytestmark = pytest.mark.gpu


def test_no_alloc_entry_matches_workspace_entry_twice(oracle):
    import torch
    from paper_2608_17641_b200 import binding as B, workloads
    assert torch.cuda.is_available()
    B.lib()
    # rows of 999 steps straddle the tiles, so the scratch (tile records, call counter) is really used
    ro = workloads.make_rollout(60, 96, 999, p_done=0.002, p_trunc=0.002)
    dev = Dev(ro)
    p = ro.params
    ws = B.Workspace(ro.N, ro.T)
    want_adv, want_ret = B.rlcs_gae(dev.rewards, dev.values, dev.dones, dev.truncs, dev.trunc_bootstrap, dev.bootstrap,
                                    gamma=p["gamma"], lam=p["lam"], workspace=ws)
    torch.cuda.synchronize()
    assert ws.device_status() == 0
    ref_adv, ref_ret = oracle.gae(ro.rewards, ro.values, ro.dones, ro.truncs, ro.trunc_bootstrap, ro.bootstrap,
                                  gamma=p["gamma"], lam=p["lam"])
    adv, ret = dev.empty_out(), dev.empty_out()
    for call in range(2):                       # the second call finds the scratch as the first one left it
        adv.fill_(float("nan"))
        ret.fill_(float("nan"))
        torch.cuda.synchronize()
        # the point of the entry point: with the outputs provided, the call takes no device memory --
        # neither from torch's caching allocator (its counters of allocation requests and of segments
        # obtained from the driver) nor from the driver directly (free bytes as cudaMemGetInfo reports
        # them; the first call on a device only looks up the built-in array's address)
        count = lambda: tuple(torch.cuda.memory_stats().get(k, 0) for k in ("allocation.all.allocated", "segment.all.allocated"))
        before, free = count(), torch.cuda.mem_get_info()[0]
        B.rlcs_gae_no_alloc(dev.rewards, dev.values, dev.dones, dev.truncs, dev.trunc_bootstrap, dev.bootstrap,
                            gamma=p["gamma"], lam=p["lam"], advantages=adv, returns=ret)
        torch.cuda.synchronize()
        assert count() == before, f"call {call} allocated device memory"
        if call == 1:
            assert torch.cuda.mem_get_info()[0] == free, "second call changed the driver's free memory"
        assert B.rlcs_no_alloc_last_device_status() == B.RLCS_OK
        for got, want, ref, name in ((adv, want_adv, ref_adv, "advantages"), (ret, want_ret, ref_ret, "returns")):
            g, w = got.cpu().numpy(), want.cpu().numpy()
            assert np.all(np.abs(g.astype(np.float64) - w) <= ATOL + RTOL * np.abs(w)), f"{name}, call {call}"
            assert_close(f"{name} vs oracle, call {call}", g, ref)


def test_no_alloc_entry_reports_a_carry_wait_that_ran_out(oracle):
    """A tile that never publishes its record makes its successor's bounded wait run out; the kernel
    still ends normally and the status reaches the caller through rlcs_no_alloc_last_device_status."""
    import torch
    from paper_2608_17641_b200 import binding as B, workloads
    ro = workloads.make_rollout(61, 4, 5000, p_done=0.0, p_trunc=0.0)      # long rows without resets: every tile needs a carry
    dev = Dev(ro)
    p = ro.params
    adv, ret = dev.empty_out(), dev.empty_out()
    call = lambda: B.rlcs_gae_no_alloc(dev.rewards, dev.values, dev.dones, dev.truncs, dev.trunc_bootstrap, dev.bootstrap,
                                       gamma=p["gamma"], lam=p["lam"], advantages=adv, returns=ret)
    call()
    assert B.rlcs_no_alloc_last_device_status() == B.RLCS_OK
    B.rlcs_debug_set_carry_fault(mute_tile=1, spin_cap=64)
    try:
        call()
        torch.cuda.synchronize()                                              # the kernel returned by itself
    finally:
        B.rlcs_debug_set_carry_fault()
    call()                                                                    # a later call does not wipe the report
    assert B.rlcs_no_alloc_last_device_status() == B.RLCS_ERR_TIMEOUT
    assert B.rlcs_no_alloc_last_device_status() == B.RLCS_OK                  # read once, then cleared
    ref_adv, _ = oracle.gae(ro.rewards, ro.values, ro.dones, ro.truncs, ro.trunc_bootstrap, ro.bootstrap,
                            gamma=p["gamma"], lam=p["lam"])
    assert_close("advantages after the timed-out call", adv.cpu().numpy(), ref_adv)


def test_no_alloc_entry_serves_any_size_that_needs_no_scratch():
    """The limit is decided on what the call uses: rows that do not straddle tiles need no records."""
    from paper_2608_17641_b200 import binding as B
    L = B.lib()
    assert L.rlcs_gae_carry_bytes(16384, 2048, 1, 1) == 0          # T is a whole number of tiles
    assert L.rlcs_workspace_bytes(16384, 2048) > L.rlcs_no_alloc_scratch_bytes()
    assert 0 < L.rlcs_gae_carry_bytes(96, 999, 1, 1) <= L.rlcs_workspace_bytes(96, 999)
    assert L.rlcs_gae_carry_bytes(64, 16384, 0, 1) == 0            # one thread-block cluster per row
    assert L.rlcs_gae_carry_bytes(64, 16384, 0, 0) > 0             # ... which needs vector access


def test_no_alloc_entry_rejects_problems_beyond_its_scratch():
    from paper_2608_17641_b200 import binding as B
    L = B.lib()
    cap = L.rlcs_no_alloc_scratch_bytes()
    assert cap == 1 << 20
    N, T = 140000, 999                          # 140 M steps in rows that straddle tiles: more records than the array holds
    assert L.rlcs_gae_carry_bytes(N, T, 0, 1) > cap
    fake = 0x7f0000000000                        # never dereferenced: the call must fail before any launch
    st = L.rlcs_gae_no_alloc(fake, fake, fake, None, None, None, fake, None, N, T, 0.99, 0.95, None)
    assert st == B.RLCS_ERR_LIMIT
    assert b"scratch" in L.rlcs_status_string(st)
