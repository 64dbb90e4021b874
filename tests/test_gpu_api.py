"""The compute_* front end (paper_2608_17641_b200.api): each call must be the binding call it stands
for, bit for bit, and the oracle's result to the parity tolerance."""
import numpy as np
import pytest

from _util import assert_close, guarded_upload, run_oracle

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2608_17641_b200 import api, binding, workloads
    binding.lib()
    binding.rlcs_debug_set_tile_variant(-1)
    return api, binding, workloads, torch


def test_front_end_matches_binding_and_oracle(oracle, env):
    api, B, W, torch = env
    ro = W.make_rollout(140, 24, 1500, p_done=0.02, p_trunc=0.01)
    p = ro.params
    up = lambda a: guarded_upload(np.ascontiguousarray(a))
    r, v, q, eq, lr, x, bv, bt = (up(getattr(ro, k)) for k in ("rewards", "values", "q_sa", "expected_q", "log_rhos", "x",
                                                                "trunc_bootstrap", "bootstrap"))
    d, tr, dany = up(ro.dones).bool(), up(ro.truncs).bool(), up(ro.any_done).bool()      # bool masks are accepted
    ref = run_oracle(oracle, ro)
    ws = B.Workspace(ro.N, ro.T)
    g = dict(gamma=p["gamma"], lam=p["lam"])
    adv, ret = api.compute_gae(r, v, d, tr, bv, bt, **g)
    a0, r0 = B.rlcs_gae(r, v, d.view(torch.uint8), tr.view(torch.uint8), bv, bt, workspace=ws, **g)
    assert torch.equal(adv, a0) and torch.equal(ret, r0)
    assert_close("gae", adv.cpu().numpy(), ref["gae"][0])
    vs, pg = api.compute_vtrace(r, v, lr, d, tr, bv, bt, gamma=p["gamma"], rho_bar=p["rho_bar"], c_bar=p["c_bar"])
    assert_close("vs", vs.cpu().numpy(), ref["vtrace"][0]); assert_close("pg", pg.cpu().numpy(), ref["vtrace"][1])
    assert_close("retrace", api.compute_retrace(r, q, eq, lr, d, tr, bv, bt, c_bar=p["c_bar"], **g).cpu().numpy(), ref["retrace"])
    assert_close("td", api.compute_td_lambda_returns(r, v, d, tr, bv, bt, **g).cpu().numpy(), ref["td_lambda"])
    assert_close("disc", api.compute_discounted_returns(r, d, tr, bv, bt, gamma=p["gamma"]).cpu().numpy(), ref["discounted_return"])
    assert_close("elig", api.compute_eligibility_traces(x, dany, **g).cpu().numpy(), ref["elig_trace"])
    assert_close("prefix", api.compute_episodic_prefix_sum(x, dany).cpu().numpy(), ref["prefix_ends_at"])
    assert_close("prefix starts_at", api.compute_episodic_prefix_sum(x, dany, boundary="starts_at").cpu().numpy(),
                 ref["prefix_starts_at"])
    # time-major and bfloat16 dispatch
    t = lambda a: a.t().contiguous()
    adv_tm, ret_tm = api.compute_gae(t(r), t(v), t(d), t(tr), t(bv), bt, time_major=True, **g)
    assert_close("gae time-major", np.ascontiguousarray(adv_tm.cpu().numpy().T), ref["gae"][0])
    h = lambda a: a.to(torch.bfloat16)
    a16, r16 = api.compute_gae(h(r), h(v), d, tr, h(bv), h(bt), **g)
    b16, _ = B.rlcs_gae_bf16(h(r), h(v), d.view(torch.uint8), tr.view(torch.uint8), h(bv), h(bt), workspace=ws, **g)
    assert a16.dtype == torch.bfloat16 and torch.equal(a16.view(torch.int16), b16.view(torch.int16))
    # normalisation, skip mask, vector traces
    nadv, nret = api.compute_gae(r, v, d, tr, bv, bt, normalize=True, **g)
    want = oracle.gae_normalized(ro.rewards, ro.values, ro.dones, ro.truncs, ro.trunc_bootstrap, ro.bootstrap, eps=1e-8, ddof=1, **g)
    assert_close("normalised adv", nadv.cpu().numpy(), want[0])
    skip = torch.rand((ro.N, ro.T), device="cuda") < 0.3
    sadv, sret, fil = api.compute_gae(r, v, d, tr, bv, bt, skip_mask=skip, **g)
    ra, rr, rf = oracle.gae_skip(ro.rewards, ro.values, ro.dones, ro.truncs, ro.trunc_bootstrap, ro.bootstrap,
                                 skip=skip.cpu().numpy().astype(np.uint8), **g)
    assert_close("skip adv", sadv.cpu().numpy(), ra)
    assert np.array_equal(fil.cpu().numpy().astype(np.float64), rf)
    xv = torch.randn((6, 200, 8), device="cuda")
    dv = torch.rand((6, 200), device="cuda") < 0.05
    assert_close("vector trace", api.compute_eligibility_traces(xv, dv, **g).cpu().numpy(),
                 oracle.elig_trace_vec(xv.cpu().numpy(), dv.cpu().numpy().astype(np.uint8), **g))
    # few long rows: the time axis is cut, the chunk records live in a cached workspace
    xl = torch.randn((4, 3000, 64), device="cuda")
    bl = torch.rand((4, 3000, 64), device="cuda") * 0.5 + 0.5
    dl = torch.rand((4, 3000), device="cuda") < 0.002
    dl8 = dl.cpu().numpy().astype(np.uint8)
    for _ in range(2):
        assert_close("long vector trace", api.compute_eligibility_traces(xl, dl, **g).cpu().numpy(),
                     oracle.elig_trace_vec(xl.cpu().numpy(), dl8, **g))
        assert_close("long vector trace, per-component decay", api.compute_eligibility_traces(xl, dl, beta=bl).cpu().numpy(),
                     oracle.elig_trace_vec_beta(xl.cpu().numpy(), bl.cpu().numpy(), dl8))
    # repeated calls reuse one workspace per shape
    before = len(api._workspaces)
    api.compute_gae(r, v, d, tr, bv, bt, **g)
    assert len(api._workspaces) == before


def test_front_end_argument_errors(env):
    api, B, W, torch = env
    r = torch.zeros((4, 8), device="cuda")
    d = torch.zeros((4, 8), dtype=torch.uint8, device="cuda")
    with pytest.raises(TypeError):
        api.compute_gae(r.double(), r.double(), d)
    with pytest.raises(ValueError):
        api.compute_gae(r.bfloat16(), r.bfloat16(), d, time_major=True)
    with pytest.raises(ValueError):
        api.compute_episodic_prefix_sum(r, d, boundary="middle")
    with pytest.raises(ValueError):
        api.compute_gae(r, r, d, normalize=True, skip_mask=d)
    with pytest.raises(ValueError):
        api.compute_eligibility_traces(r, d, beta=r)
    with pytest.raises(TypeError):
        api.compute_gae(r.cpu(), r.cpu(), d.cpu())               # there is no CPU path


def test_prepared_calls_repeat_the_direct_call(env, oracle):
    """binding.prepare(): arguments marshalled once, then only the C call -- same bits as the wrapper."""
    api, B, W, torch = env
    ro = W.make_rollout(130, 48, 999, p_done=0.01, p_trunc=0.01)
    up = lambda a: guarded_upload(a)
    r, v, d, tr, bv, bt = up(ro.rewards), up(ro.values), up(ro.dones), up(ro.truncs), up(ro.trunc_bootstrap), up(ro.bootstrap)
    ws = B.Workspace(ro.N, ro.T)
    want_adv, want_ret = B.rlcs_gae(r, v, d, tr, bv, bt, gamma=0.99, lam=0.95, workspace=ws)
    step = B.prepare(B.rlcs_gae, r, v, d, tr, bv, bt, gamma=0.99, lam=0.95, workspace=ws)
    adv, ret = step.outputs
    adv.fill_(float("nan"))
    for _ in range(3):
        out = step()
        assert out[0] is adv
    torch.cuda.synchronize()
    assert torch.equal(adv, want_adv) and torch.equal(ret, want_ret) and ws.device_status() == 0
    # a wrapper that makes three launches and creates its own workspace
    norm = B.prepare(B.rlcs_gae_normalized, r, v, d, tr, bv, bt, gamma=0.99, lam=0.95, eps=1e-8, ddof=1)
    assert len(norm._calls) == 1
    nadv, _ = norm()
    torch.cuda.synchronize()
    want, _ = B.rlcs_gae_normalized(r, v, d, tr, bv, bt, gamma=0.99, lam=0.95, eps=1e-8, ddof=1)
    assert torch.equal(nadv, want)
    # on an explicit stream handle
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    adv.fill_(0)
    torch.cuda.synchronize()
    step(s.cuda_stream)
    s.synchronize()
    assert torch.equal(adv, want_adv)
