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
    # rows of 1000 steps straddle the tiles, so the scratch (tile records, call counter) is really used
    ro = workloads.make_rollout(60, 96, 1000, p_done=0.002, p_trunc=0.002)
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
        B.rlcs_gae_no_alloc(dev.rewards, dev.values, dev.dones, dev.truncs, dev.trunc_bootstrap, dev.bootstrap,
                            gamma=p["gamma"], lam=p["lam"], advantages=adv, returns=ret)
        torch.cuda.synchronize()
        for got, want, ref, name in ((adv, want_adv, ref_adv, "advantages"), (ret, want_ret, ref_ret, "returns")):
            g, w = got.cpu().numpy(), want.cpu().numpy()
            assert np.all(np.abs(g.astype(np.float64) - w) <= ATOL + RTOL * np.abs(w)), f"{name}, call {call}"
            assert_close(f"{name} vs oracle, call {call}", g, ref)


def test_no_alloc_entry_rejects_problems_beyond_its_scratch():
    from paper_2608_17641_b200 import binding as B
    L = B.lib()
    cap = L.rlcs_no_alloc_scratch_bytes()
    assert cap == 1 << 20
    N, T = 40000, 1000                           # 40 M steps: needs more tile records than the array holds
    assert L.rlcs_workspace_bytes(N, T) > cap
    fake = 0x7f0000000000                        # never dereferenced: the call must fail before any launch
    st = L.rlcs_gae_no_alloc(fake, fake, fake, None, None, None, fake, None, N, T, 0.99, 0.95, None)
    assert st == B.RLCS_ERR_LIMIT
    assert b"scratch" in L.rlcs_status_string(st)
