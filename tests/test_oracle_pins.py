"""Pins for the CPU oracle: what the paper and the mathematics fix, not the oracle's own formulas.

The brute force below takes Table 1's (alpha_t, beta_t, carry) literally -- multiplicative
(1 - d) masks, bootstrap rules of Section 3.2 / 3.3.4 -- and evaluates the explicit O(T^2) sum
    A_t = sum_{k>=t} (prod_{j=t}^{k-1} beta_j) alpha_k + (prod_{j=t}^{T-1} beta_j) A_T
(or its forward mirror).  The oracle is a branchy sequential recurrence; the two share no code.
"""
import os

import numpy as np
import pytest

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------------------- brute force
def explicit_sum_backward(alpha, beta, carry):
    T = len(alpha)
    A = np.zeros(T)
    for t in range(T):
        acc, prod = 0.0, 1.0
        for k in range(t, T):
            acc += prod * alpha[k]
            prod *= beta[k]
        A[t] = acc + prod * carry
    return A


def explicit_sum_forward(alpha, beta):
    T = len(alpha)
    A = np.zeros(T)
    for t in range(T):
        acc, prod = 0.0, 1.0
        for k in range(t, -1, -1):
            acc += prod * alpha[k]
            prod *= beta[k]
        A[t] = acc          # A_{-1} = 0
    return A


def _row_inputs(rng, T, p_flag):
    f = lambda: rng.standard_normal(T).astype(np.float32)
    term = (rng.random(T) < p_flag).astype(np.uint8)
    trunc = (rng.random(T) < p_flag).astype(np.uint8)
    return dict(r=f(), V=f(), q=f(), eq=f(), lr=(0.5 * rng.standard_normal(T)).astype(np.float32),
                x=f(), bv=f(), term=term, trunc=trunc, boot=np.float32(rng.standard_normal()))


def _table1_successor(X, i, t, T):
    """(1 - d^term_t) * [continuation value of step t]: bv at a truncation, the window-edge
    bootstrap at a non-truncated t = T-1, the stored X[t+1] otherwise."""
    term, trunc = float(i["term"][t]), i["trunc"][t]
    if trunc:
        nxt = float(i["bv"][t])
    elif t == T - 1:
        nxt = float(i["boot"])
    else:
        nxt = float(X[t + 1])
    return (1.0 - term) * nxt


def table1_gae(i, g, l):
    T = len(i["r"])
    d = np.maximum(i["term"], i["trunc"]).astype(float)
    alpha = np.array([float(i["r"][t]) + g * _table1_successor(i["V"], i, t, T) - float(i["V"][t])
                      for t in range(T)])
    beta = g * l * (1.0 - d)
    return explicit_sum_backward(alpha, beta, 0.0)


def table1_td_lambda(i, g, l):
    T = len(i["r"])
    d = np.maximum(i["term"], i["trunc"]).astype(float)
    alpha = np.zeros(T)
    for t in range(T):
        s = _table1_successor(i["V"], i, t, T)
        # Section 3.3.4: at a truncated step the continuation enters alpha with the full gamma.
        alpha[t] = float(i["r"][t]) + (g * s if i["trunc"][t] else g * (1.0 - l) * s)
    beta = g * l * (1.0 - d)
    return explicit_sum_backward(alpha, beta, float(i["boot"]))


def table1_discounted(i, g):
    T = len(i["r"])
    d = np.maximum(i["term"], i["trunc"]).astype(float)
    alpha = np.array([float(i["r"][t]) + (g * (1.0 - float(i["term"][t])) * float(i["bv"][t])
                                          if i["trunc"][t] else 0.0) for t in range(T)])
    beta = g * (1.0 - d)
    return explicit_sum_backward(alpha, beta, float(i["boot"]))


def table1_vtrace(i, g, rho_bar, c_bar):
    T = len(i["r"])
    d = np.maximum(i["term"], i["trunc"]).astype(float)
    raw = np.exp(i["lr"].astype(float))
    rho, c = np.minimum(rho_bar, raw), np.minimum(c_bar, raw)
    alpha = np.array([rho[t] * (float(i["r"][t]) + g * _table1_successor(i["V"], i, t, T) - float(i["V"][t]))
                      for t in range(T)])
    beta = g * c * (1.0 - d)
    vs = explicit_sum_backward(alpha, beta, 0.0) + i["V"].astype(float)
    adv = np.zeros(T)
    for t in range(T):
        if d[t] or t == T - 1:
            vn = _table1_successor(i["V"], i, t, T)
        else:
            vn = vs[t + 1]
        adv[t] = rho[t] * (float(i["r"][t]) + g * vn - float(i["V"][t]))
    return vs, adv


def table1_retrace(i, g, l, c_bar):
    T = len(i["r"])
    d = np.maximum(i["term"], i["trunc"]).astype(float)
    c = l * np.minimum(c_bar, np.exp(i["lr"].astype(float)))
    c_shift = np.append(c[1:], 0.0)          # c_{t+1}, with c_T = 0
    alpha = np.array([float(i["r"][t]) + g * _table1_successor(i["eq"], i, t, T) - float(i["q"][t])
                      for t in range(T)])
    beta = g * c_shift * (1.0 - d)
    return explicit_sum_backward(alpha, beta, 0.0) + i["q"].astype(float)


def table1_forward(i, decay, starts_at=False):
    T = len(i["x"])
    d = np.maximum(i["term"], i["trunc"]).astype(float)
    d_prev = np.append(0.0, d[:-1])          # d_{-1} := 0
    beta = decay * (1.0 - (d if starts_at else d_prev))
    return explicit_sum_forward(i["x"].astype(float), beta)


def _call(oracle, name, i, **kw):
    two = lambda a: None if a is None else np.asarray(a)[None, :]
    common = dict(dones=two(i["term"]), truncs=two(i["trunc"]), trunc_bootstrap=two(i["bv"]),
                  bootstrap=np.array([i["boot"]], np.float32))
    if name == "gae":
        return oracle.gae(two(i["r"]), two(i["V"]), **common, **kw)
    if name == "td":
        return oracle.td_lambda(two(i["r"]), two(i["V"]), **common, **kw)
    if name == "disc":
        return oracle.discounted_return(two(i["r"]), **common, **kw)
    if name == "vtrace":
        return oracle.vtrace(two(i["r"]), two(i["V"]), two(i["lr"]), **common, **kw)
    if name == "retrace":
        return oracle.retrace(two(i["r"]), two(i["q"]), two(i["eq"]), two(i["lr"]), **common, **kw)
    raise KeyError(name)


G32, L32 = float(np.float32(0.99)), float(np.float32(0.95))


# ----------------------------------------------------------------------------- P3: Table 1 brute force
@pytest.mark.parametrize("T", [1, 2, 3, 5, 17, 40])
@pytest.mark.parametrize("p_flag", [0.0, 0.1, 0.5])
def test_table1_explicit_sum_all_algorithms(oracle, T, p_flag):
    rng = np.random.default_rng(1000 * T + int(100 * p_flag))
    for _ in range(6):
        i = _row_inputs(rng, T, p_flag)
        if T > 1 and rng.random() < 0.5:      # force flags at both ends and a term AND trunc step
            i["trunc"][T - 1] = 1
            i["term"][0] = 1
            i["term"][T // 2] = i["trunc"][T // 2] = 1
        adv, ret = _call(oracle, "gae", i, gamma=0.99, lam=0.95)
        np.testing.assert_allclose(adv[0], table1_gae(i, G32, L32), rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(ret[0], table1_gae(i, G32, L32) + i["V"], rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(_call(oracle, "td", i, gamma=0.99, lam=0.95)[0],
                                   table1_td_lambda(i, G32, L32), rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(_call(oracle, "disc", i, gamma=0.99)[0],
                                   table1_discounted(i, G32), rtol=1e-12, atol=1e-12)
        for rb, cb in [(1.0, 1.0), (1.5, 0.75)]:
            vs, pg = _call(oracle, "vtrace", i, gamma=0.99, rho_bar=rb, c_bar=cb)
            evs, epg = table1_vtrace(i, G32, float(np.float32(rb)), float(np.float32(cb)))
            np.testing.assert_allclose(vs[0], evs, rtol=1e-12, atol=1e-12)
            np.testing.assert_allclose(pg[0], epg, rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(_call(oracle, "retrace", i, gamma=0.99, lam=0.95, c_bar=1.0)[0],
                                   table1_retrace(i, G32, L32, 1.0), rtol=1e-12, atol=1e-12)
        d = np.maximum(i["term"], i["trunc"])[None, :]
        np.testing.assert_allclose(oracle.elig_trace(i["x"][None, :], d, gamma=0.99, lam=0.95)[0],
                                   table1_forward(i, G32 * L32), rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(oracle.episodic_prefix_sum(i["x"][None, :], d)[0],
                                   table1_forward(i, 1.0), rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(oracle.episodic_prefix_sum(i["x"][None, :], d, starts_at=True)[0],
                                   table1_forward(i, 1.0, starts_at=True), rtol=1e-12, atol=1e-12)


def test_absent_truncs_and_bootstrap_equal_zero_filled(oracle):
    """HAS_TRUNCATIONS=False / HAS_BOOTSTRAP=False (Section 4.2) = all-false mask / zero vector."""
    rng = np.random.default_rng(7)
    N, T = 5, 33
    r, V = rng.standard_normal((2, N, T)).astype(np.float32)
    d = (rng.random((N, T)) < 0.1).astype(np.uint8)
    z8, zf, zb = np.zeros((N, T), np.uint8), np.ones((N, T), np.float32), np.zeros(N, np.float32)
    a0, r0 = oracle.gae(r, V, d, gamma=0.9, lam=0.8)
    a1, r1 = oracle.gae(r, V, d, z8, zf, zb, gamma=0.9, lam=0.8)
    assert np.array_equal(a0, a1) and np.array_equal(r0, r1)
    assert np.array_equal(oracle.discounted_return(r, d, gamma=0.9),
                          oracle.discounted_return(r, d, z8, zf, zb, gamma=0.9))


# ----------------------------------------------------------------------------- P1 / P2: the operator
def test_combine_associative_on_random_triples(oracle):
    rng = np.random.default_rng(1)
    for _ in range(200):
        C, B, A = rng.standard_normal((3, 2))
        left = oracle.combine(oracle.combine(C, B), A)
        right = oracle.combine(C, oracle.combine(B, A))
        np.testing.assert_allclose(left, right, rtol=1e-12, atol=1e-12)
        # closed form of the proof of Proposition 1
        np.testing.assert_allclose(left, (C[0] + C[1] * B[0] + B[1] * C[1] * A[0], A[1] * B[1] * C[1]),
                                   rtol=1e-12, atol=1e-12)


def test_severing_identity(oracle):
    """(alpha_t, 0) (+) X = (alpha_t, 0) for any X (Section 5.2)."""
    rng = np.random.default_rng(2)
    for _ in range(50):
        a, xa, xb = rng.standard_normal(3) * 1e3
        assert oracle.combine((a, 0.0), (xa, xb)) == (a, 0.0)


def _golden_exprs():
    out = {}
    with open(os.path.join(GOLDEN, "four_step_trace.txt")) as fh:
        for line in fh:
            line = line.strip()
            if line and not line.startswith("#"):
                k, v = line.split("=", 1)
                out[k.strip()] = v.strip()
    return out


def test_four_step_expansion_and_appendix_trace(oracle):
    """The 4-step expansion (Section 5.1) and every intermediate tuple of Appendix A."""
    ex = _golden_exprs()
    rng = np.random.default_rng(3)
    for _ in range(20):
        a, b = rng.standard_normal((2, 4))
        ns = {f"a{k}": a[k] for k in range(4)} | {f"b{k}": b[k] for k in range(4)}
        val = lambda name: eval(ex[name], {"__builtins__": {}}, ns)
        A = oracle.linear_recurrence(a, b, 0.0)
        np.testing.assert_allclose(A[0], val("A0"), rtol=1e-13)
        T = {k: (a[4 - k], b[4 - k]) for k in (1, 2, 3, 4)}      # thread k holds timestep 4-k
        T12 = oracle.combine(T[2], T[1])
        T23 = oracle.combine(T[3], T[2])
        T34 = oracle.combine(T[4], T[3])
        T14 = oracle.combine(T34, T12)
        T13 = oracle.combine(T23, T[1])
        for name, tup in (("T11", T[1]), ("T12", T12), ("T23", T23), ("T34", T34), ("T14", T14)):
            np.testing.assert_allclose(tup, (val(name + ".alpha"), val(name + ".beta")), rtol=1e-13)
        # each thread's final tuple's alpha is the recurrence value at its timestep (carry 0)
        np.testing.assert_allclose([T14[0], T13[0], T12[0], T[1][0]], A, rtol=1e-13)
        # forward mirror: A_t = alpha_t + beta_t A_{t-1}
        F = oracle.linear_recurrence(a, b, 0.0, forward=True)
        np.testing.assert_allclose(F[3], a[3] + b[3] * (a[2] + b[2] * (a[1] + b[1] * a[0])), rtol=1e-13)


# ----------------------------------------------------------------------------- special cases / identities
def _batch(seed, N=6, T=50, p=0.08):
    rng = np.random.default_rng(seed)
    f = lambda *s: rng.standard_normal(s or (N, T)).astype(np.float32)
    return dict(r=f(), V=f(), q=f(), eq=f(), lr=(0.5 * f()).astype(np.float32), x=f(), bv=f(),
                term=(rng.random((N, T)) < p).astype(np.uint8), trunc=(rng.random((N, T)) < p).astype(np.uint8),
                boot=f(N))


def _bk(b):
    return dict(dones=b["term"], truncs=b["trunc"], trunc_bootstrap=b["bv"], bootstrap=b["boot"])


def test_gamma_zero_gives_alpha(oracle):
    b = _batch(11)
    r, V = b["r"].astype(float), b["V"].astype(float)
    adv, ret = oracle.gae(b["r"], b["V"], **_bk(b), gamma=0.0, lam=0.95)
    np.testing.assert_array_equal(adv, r - V)
    np.testing.assert_array_equal(oracle.td_lambda(b["r"], b["V"], **_bk(b), gamma=0.0, lam=0.95), r)
    np.testing.assert_array_equal(oracle.discounted_return(b["r"], **_bk(b), gamma=0.0), r)
    vs, pg = oracle.vtrace(b["r"], b["V"], b["lr"], **_bk(b), gamma=0.0)
    rho = np.minimum(1.0, np.exp(b["lr"].astype(float)))
    np.testing.assert_allclose(vs, V + rho * (r - V), rtol=1e-14)
    np.testing.assert_allclose(pg, rho * (r - V), rtol=1e-14)
    np.testing.assert_array_equal(oracle.retrace(b["r"], b["q"], b["eq"], b["lr"], **_bk(b), gamma=0.0, lam=0.9),
                                  b["q"].astype(float) + (r - b["q"].astype(float)))
    d = np.maximum(b["term"], b["trunc"])
    np.testing.assert_array_equal(oracle.elig_trace(b["x"], d, gamma=0.0, lam=0.9), b["x"].astype(float))


def test_gae_lambda_zero_is_one_step_td(oracle):
    b = _batch(12)
    N, T = b["r"].shape
    adv, _ = oracle.gae(b["r"], b["V"], **_bk(b), gamma=0.99, lam=0.0)
    Vn = np.concatenate([b["V"][:, 1:], b["boot"][:, None]], axis=1).astype(float)
    Vn = np.where(b["trunc"] != 0, b["bv"].astype(float), Vn)
    Vn = np.where(b["term"] != 0, 0.0, Vn)
    np.testing.assert_allclose(adv, b["r"] + G32 * Vn - b["V"], rtol=1e-13, atol=1e-13)


def test_gae_lambda_one_is_return_minus_value(oracle):
    b = _batch(13)
    adv, ret = oracle.gae(b["r"], b["V"], **_bk(b), gamma=0.99, lam=1.0)
    G = oracle.discounted_return(b["r"], **_bk(b), gamma=0.99)
    np.testing.assert_allclose(adv, G - b["V"], rtol=1e-11, atol=1e-11)
    np.testing.assert_allclose(ret, G, rtol=1e-11, atol=1e-11)


@pytest.mark.parametrize("lam", [0.0, 0.3, 0.95, 1.0])
def test_td_lambda_minus_value_is_gae(oracle, lam):
    b = _batch(14)
    adv, ret = oracle.gae(b["r"], b["V"], **_bk(b), gamma=0.99, lam=lam)
    G = oracle.td_lambda(b["r"], b["V"], **_bk(b), gamma=0.99, lam=lam)
    np.testing.assert_allclose(G - b["V"], adv, rtol=1e-11, atol=1e-11)
    np.testing.assert_allclose(G, ret, rtol=1e-11, atol=1e-11)


def test_td_lambda_window_edge_independent_of_lambda(oracle):
    """G_{T-1} = r_{T-1} + gamma V(s_T) for every lambda when the last step carries no flag."""
    b = _batch(15)
    b["term"][:, -1] = 0
    b["trunc"][:, -1] = 0
    for lam in (0.0, 0.5, 1.0):
        G = oracle.td_lambda(b["r"], b["V"], **_bk(b), gamma=0.99, lam=lam)
        np.testing.assert_allclose(G[:, -1], b["r"][:, -1] + G32 * b["boot"].astype(float), rtol=1e-14)


def test_vtrace_on_policy_reduces_to_discounted_return(oracle):
    b = _batch(16)
    zero = np.zeros_like(b["lr"])
    vs, pg = oracle.vtrace(b["r"], b["V"], zero, **_bk(b), gamma=0.99)
    G = oracle.discounted_return(b["r"], **_bk(b), gamma=0.99)
    np.testing.assert_allclose(vs, G, rtol=1e-11, atol=1e-11)
    # with rho = c = 1 the advantage is r + gamma v_{t+1} - V = vs - V
    np.testing.assert_allclose(pg, G - b["V"], rtol=1e-11, atol=1e-11)


def test_vtrace_equal_clips_make_advantage_the_delta(oracle):
    """With rho_bar = c_bar, rho_t = c_t and A_t = rho_t(r + gamma v_{t+1} - V) = Delta_t = vs - V."""
    b = _batch(17)
    vs, pg = oracle.vtrace(b["r"], b["V"], b["lr"], **_bk(b), gamma=0.99, rho_bar=0.8, c_bar=0.8)
    np.testing.assert_allclose(pg, vs - b["V"], rtol=1e-11, atol=1e-11)


def test_retrace_with_value_inputs_is_gae(oracle):
    b = _batch(18)
    zero = np.zeros_like(b["lr"])
    tgt = oracle.retrace(b["r"], b["V"], b["V"], zero, **_bk(b), gamma=0.99, lam=0.95)
    adv, _ = oracle.gae(b["r"], b["V"], **_bk(b), gamma=0.99, lam=0.95)
    np.testing.assert_allclose(tgt - b["V"], adv, rtol=1e-11, atol=1e-11)


def test_retrace_lambda1_matches_vtrace_trace_coefficient_shifted(oracle):
    """Index shift: Retrace's Delta_t depends on log_rho[t+1], not on log_rho[t]; V-Trace's the opposite."""
    b = _batch(19, N=1, T=12, p=0.0)
    base = oracle.retrace(b["r"], b["q"], b["eq"], b["lr"], **_bk(b), gamma=0.99, lam=0.9)
    lr2 = b["lr"].copy()
    lr2[0, 0] -= 1.0                                  # first column never enters Retrace
    assert np.array_equal(base, oracle.retrace(b["r"], b["q"], b["eq"], lr2, **_bk(b), gamma=0.99, lam=0.9))
    lr3 = b["lr"].copy()
    lr3[0, 5] -= 1.0                                  # c_5 scales Delta_5 inside Delta_4
    out3 = oracle.retrace(b["r"], b["q"], b["eq"], lr3, **_bk(b), gamma=0.99, lam=0.9)
    assert out3[0, 4] != base[0, 4] and np.array_equal(out3[0, 5:], base[0, 5:])
    v0, _ = oracle.vtrace(b["r"], b["V"], b["lr"], **_bk(b), gamma=0.99)
    v3, _ = oracle.vtrace(b["r"], b["V"], lr3, **_bk(b), gamma=0.99)
    assert v3[0, 5] != v0[0, 5] and np.array_equal(v3[0, 6:], v0[0, 6:])


def test_retrace_expected_q_column0_never_read(oracle):
    b = _batch(20)
    base = oracle.retrace(b["r"], b["q"], b["eq"], b["lr"], **_bk(b), gamma=0.99, lam=0.9)
    eq2 = b["eq"].copy()
    eq2[:, 0] = 1e6
    assert np.array_equal(base, oracle.retrace(b["r"], b["q"], eq2, b["lr"], **_bk(b), gamma=0.99, lam=0.9))


# ----------------------------------------------------------------------------- closed forms
def test_constant_reward_geometric_closed_form(oracle):
    T, c, boot, g = 60, 0.7, -1.3, 0.9
    g32 = float(np.float32(g))
    r = np.full((1, T), c, np.float32)
    G = oracle.discounted_return(r, np.zeros((1, T), np.uint8), bootstrap=np.array([boot], np.float32), gamma=g)
    k = T - np.arange(T)
    c32, b32 = float(np.float32(c)), float(np.float32(boot))
    np.testing.assert_allclose(G[0], c32 * (1 - g32 ** k) / (1 - g32) + g32 ** k * b32, rtol=1e-12)


def test_bootstrap_priced_once(oracle):
    """r = 0, V = 0, boot = b: GAE A_t = gamma b (gamma lambda)^{T-1-t} (carry 0, bootstrap only in
    alpha_{T-1}); TD(lambda) gives the same; discounted return gamma^{T-t} b.  Seeding the GAE carry
    with b instead would add b (gamma lambda)^{T-t} at every step."""
    T, b, g, l = 25, 2.5, 0.99, 0.95
    z = np.zeros((1, T), np.float32)
    d = np.zeros((1, T), np.uint8)
    bt = np.array([b], np.float32)
    k = T - 1 - np.arange(T)
    adv, _ = oracle.gae(z, z, d, bootstrap=bt, gamma=g, lam=l)
    np.testing.assert_allclose(adv[0], G32 * b * (G32 * L32) ** k, rtol=1e-12)
    np.testing.assert_allclose(oracle.td_lambda(z, z, d, bootstrap=bt, gamma=g, lam=l)[0],
                               G32 * b * (G32 * L32) ** k, rtol=1e-12)
    np.testing.assert_allclose(oracle.discounted_return(z, d, bootstrap=bt, gamma=g)[0],
                               G32 ** (k + 1) * b, rtol=1e-12)


def test_forward_scans_constant_input_closed_form(oracle):
    T, c = 40, 0.5
    x = np.full((1, T), c, np.float32)
    d = np.zeros((1, T), np.uint8)
    d[0, [6, 7, 20]] = 1
    k = np.zeros(T)                                   # steps since the segment started
    for t in range(1, T):
        k[t] = 0 if d[0, t - 1] else k[t - 1] + 1
    gl = G32 * L32
    np.testing.assert_allclose(oracle.elig_trace(x, d, gamma=0.99, lam=0.95)[0],
                               c * (1 - gl ** (k + 1)) / (1 - gl), rtol=1e-12)
    np.testing.assert_array_equal(oracle.episodic_prefix_sum(x, d)[0], c * (k + 1))
    ks = np.zeros(T)                                  # starts_at: the flagged step opens the segment
    for t in range(1, T):
        ks[t] = 0 if d[0, t] else ks[t - 1] + 1
    np.testing.assert_array_equal(oracle.episodic_prefix_sum(x, d, starts_at=True)[0], c * (ks + 1))


def test_prefix_sum_without_flags_is_cumsum(oracle):
    rng = np.random.default_rng(21)
    x = rng.standard_normal((3, 100)).astype(np.float32)
    d = np.zeros((3, 100), np.uint8)
    np.testing.assert_allclose(oracle.episodic_prefix_sum(x, d), np.cumsum(x.astype(np.float64), axis=1), rtol=1e-13)


def test_sparse_terminal_reward_gamma_one_is_exact(oracle):
    """gamma = 1, reward only at segment ends: every G_t in a closed segment equals that segment's
    terminal reward exactly; in the last open segment it equals r_{T-1} + boot."""
    from paper_2608_17641_b200 import workloads
    ro = workloads.config4(N=4, T=3000)
    G = oracle.discounted_return(ro.rewards, ro.dones, bootstrap=ro.bootstrap, gamma=1.0)
    for n in range(ro.N):
        ends = list(np.flatnonzero(ro.dones[n])) + [ro.T - 1]
        start = 0
        for e in ends:
            want = float(ro.rewards[n, e])
            if e == ro.T - 1 and not ro.dones[n, e]:
                want += float(ro.bootstrap[n])
            assert np.all(G[n, start:e + 1] == want)
            start = e + 1


# ----------------------------------------------------------------------------- segmentation
def test_severed_steps_equal_alpha_exactly(oracle):
    b = _batch(22)
    d = (b["term"] != 0) | (b["trunc"] != 0)
    tm = b["term"] != 0
    G = oracle.discounted_return(b["r"], **_bk(b), gamma=0.99)
    assert np.array_equal(G[tm], b["r"].astype(float)[tm])
    adv, _ = oracle.gae(b["r"], b["V"], **_bk(b), gamma=0.99, lam=0.95)
    assert np.array_equal(adv[tm], (b["r"].astype(float) - b["V"].astype(float))[tm])
    tr_only = (b["trunc"] != 0) & ~tm
    assert np.array_equal(G[tr_only], (b["r"].astype(float) + G32 * b["bv"].astype(float))[tr_only])
    assert d.any()


def test_segment_isolation(oracle):
    """Changing inputs after a flagged step never changes outputs at or before it (backward scans),
    and changing inputs before it never changes outputs after it (forward scans)."""
    b = _batch(23, N=1, T=64, p=0.0)
    b["term"][0, 30] = 1
    base_adv, _ = oracle.gae(b["r"], b["V"], **_bk(b), gamma=0.99, lam=0.95)
    base_vs, _ = oracle.vtrace(b["r"], b["V"], b["lr"], **_bk(b), gamma=0.99)
    b2 = {k: (v.copy() if isinstance(v, np.ndarray) else v) for k, v in b.items()}
    for key in ("r", "V", "lr", "bv"):
        b2[key][0, 31:] += 5.0
    b2["boot"] = b["boot"] + 3.0
    adv2, _ = oracle.gae(b2["r"], b2["V"], **_bk(b2), gamma=0.99, lam=0.95)
    vs2, _ = oracle.vtrace(b2["r"], b2["V"], b2["lr"], **_bk(b2), gamma=0.99)
    assert np.array_equal(adv2[0, :31], base_adv[0, :31]) and not np.array_equal(adv2[0, 31:], base_adv[0, 31:])
    assert np.array_equal(vs2[0, :31], base_vs[0, :31])
    d = b["term"]
    z0 = oracle.elig_trace(b["x"], d, gamma=0.99, lam=0.95)
    x2 = b["x"].copy()
    x2[0, :31] += 5.0
    z2 = oracle.elig_trace(x2, d, gamma=0.99, lam=0.95)
    assert np.array_equal(z2[0, 31:], z0[0, 31:]) and not np.array_equal(z2[0, :31], z0[0, :31])


def test_truncated_last_step_uses_truncation_value_not_window_bootstrap(oracle):
    b = _batch(24, p=0.0)
    b["trunc"][:, -1] = 1
    kw = _bk(b)
    fns = [lambda **k: oracle.gae(b["r"], b["V"], gamma=0.99, lam=0.95, **k)[0],
           lambda **k: oracle.td_lambda(b["r"], b["V"], gamma=0.99, lam=0.95, **k),
           lambda **k: oracle.discounted_return(b["r"], gamma=0.99, **k),
           lambda **k: oracle.vtrace(b["r"], b["V"], b["lr"], gamma=0.99, **k)[0],
           lambda **k: oracle.retrace(b["r"], b["q"], b["eq"], b["lr"], gamma=0.99, lam=0.95, **k)]
    for fn in fns:
        base = fn(**kw)
        other_boot = dict(kw, bootstrap=b["boot"] + 1.0)
        assert np.array_equal(fn(**other_boot), base)
        bv2 = b["bv"].copy()
        bv2[:, -1] += 1.0
        assert not np.array_equal(fn(**dict(kw, trunc_bootstrap=bv2)), base)


def test_termination_wins_over_truncation(oracle):
    b = _batch(25, p=0.0)
    b["term"][:, 10] = 1
    base, _ = oracle.gae(b["r"], b["V"], **_bk(b), gamma=0.99, lam=0.95)
    b["trunc"][:, 10] = 1
    both, _ = oracle.gae(b["r"], b["V"], **_bk(b), gamma=0.99, lam=0.95)
    assert np.array_equal(base, both)


def test_nonbinary_flags_count_as_true(oracle):
    b = _batch(26)
    base = oracle.discounted_return(b["r"], **_bk(b), gamma=0.99)
    kw = _bk(b)
    kw["dones"] = b["term"] * np.uint8(255)
    kw["truncs"] = b["trunc"] * np.uint8(2)
    assert np.array_equal(oracle.discounted_return(b["r"], **kw, gamma=0.99), base)


def test_single_step_rows(oracle):
    """T = 1: GAE gives r + gamma*successor - V."""
    r = np.array([[1.0], [2.0], [3.0]], np.float32)
    V = np.array([[0.5], [0.25], [0.125]], np.float32)
    term = np.array([[0], [1], [0]], np.uint8)
    trunc = np.array([[0], [0], [1]], np.uint8)
    bv = np.array([[9.0], [9.0], [4.0]], np.float32)
    boot = np.array([2.0, 7.0, 7.0], np.float32)
    adv, ret = oracle.gae(r, V, term, trunc, bv, boot, gamma=0.5, lam=0.95)
    np.testing.assert_array_equal(adv[:, 0], [1.0 + 0.5 * 2.0 - 0.5, 2.0 - 0.25, 3.0 + 0.5 * 4.0 - 0.125])
    np.testing.assert_array_equal(ret[:, 0], adv[:, 0] + V[:, 0])


def test_hand_worked_three_step_example(oracle):
    """r = 1, V = 0, gamma = 0.5, lambda = 1, no flags, no bootstrap: A = [1.75, 1.5, 1] by hand;
    a termination at t = 1 gives [1.5, 1, 1]."""
    r = np.ones((1, 3), np.float32)
    z = np.zeros((1, 3), np.float32)
    d = np.zeros((1, 3), np.uint8)
    np.testing.assert_array_equal(oracle.gae(r, z, d, gamma=0.5, lam=1.0)[0][0], [1.75, 1.5, 1.0])
    d[0, 1] = 1
    np.testing.assert_array_equal(oracle.gae(r, z, d, gamma=0.5, lam=1.0)[0][0], [1.5, 1.0, 1.0])
    np.testing.assert_array_equal(oracle.elig_trace(r, d, gamma=0.5, lam=1.0)[0], [1.0, 1.5, 1.0])


def test_rows_parallel_helper_matches_single_call(oracle):
    b = _batch(27, N=13, T=40)
    one = oracle.gae(b["r"], b["V"], **_bk(b), gamma=0.99, lam=0.95)
    par = oracle.run_rows_parallel(
        oracle.gae, dict(rewards=b["r"], values=b["V"], dones=b["term"], truncs=b["trunc"],
                         trunc_bootstrap=b["bv"]), dict(bootstrap=b["boot"]), threads=4, gamma=0.99, lam=0.95)
    assert np.array_equal(one[0], par[0]) and np.array_equal(one[1], par[1])


# ----------------------------------------------------------------------------- advantage normalisation
def test_normalised_advantages_hand_example(oracle):
    """r = [1, 2, 3], V = 0, gamma = 0: A = r.  mean 2; population std sqrt(2/3), sample std 1."""
    r = np.array([[1.0, 2.0, 3.0]], np.float32)
    z = np.zeros((1, 3), np.float32)
    d = np.zeros((1, 3), np.uint8)
    a0, ret = oracle.gae_normalized(r, z, d, gamma=0.0, lam=0.9, eps=0.0, ddof=0)
    np.testing.assert_allclose(a0[0], [-np.sqrt(1.5), 0.0, np.sqrt(1.5)], rtol=1e-14)
    a1, _ = oracle.gae_normalized(r, z, d, gamma=0.0, lam=0.9, eps=0.0, ddof=1)
    np.testing.assert_allclose(a1[0], [-1.0, 0.0, 1.0], rtol=1e-14)
    np.testing.assert_array_equal(ret[0], [1.0, 2.0, 3.0])         # returns stay un-normalised


def test_normalised_advantages_match_library_mean_and_std(oracle):
    b = _batch(31, N=9, T=77)
    for ddof in (0, 1):
        for eps in (0.0, 1e-8, 0.5):
            out, ret = oracle.gae_normalized(b["r"], b["V"], **_bk(b), gamma=0.99, lam=0.95, eps=eps, ddof=ddof)
            adv, ret0 = oracle.gae(b["r"], b["V"], **_bk(b), gamma=0.99, lam=0.95)
            want = (adv - np.mean(adv)) / (np.std(adv, ddof=ddof) + float(np.float32(eps)))
            np.testing.assert_allclose(out, want, rtol=1e-12, atol=1e-12)
            assert np.array_equal(ret, ret0)
            if eps == 0.0:
                assert abs(out.mean()) < 1e-12
                np.testing.assert_allclose(out.std(ddof=ddof), 1.0, rtol=1e-12)


def test_normalised_advantages_scale_invariance_and_degenerate_cases(oracle):
    """GAE is linear in (rewards, values, bootstraps): scaling them by c > 0 leaves the normalised
    advantages unchanged (eps = 0).  A constant advantage gives zeros; so does a single step."""
    b = _batch(32, N=4, T=60)
    base, _ = oracle.gae_normalized(b["r"], b["V"], **_bk(b), gamma=0.99, lam=0.95, eps=0.0, ddof=1)
    kw = _bk(b)
    kw["trunc_bootstrap"] = b["bv"] * np.float32(4.0)
    kw["bootstrap"] = b["boot"] * np.float32(4.0)
    scaled, _ = oracle.gae_normalized(b["r"] * np.float32(4.0), b["V"] * np.float32(4.0), **kw, gamma=0.99, lam=0.95,
                                      eps=0.0, ddof=1)
    np.testing.assert_allclose(scaled, base, rtol=1e-10, atol=1e-12)
    ones = np.ones((3, 5), np.float32)
    const, _ = oracle.gae_normalized(ones, np.zeros_like(ones), np.ones((3, 5), np.uint8), gamma=0.9, lam=0.9, eps=1e-8)
    assert np.array_equal(const, np.zeros((3, 5)))
    single, _ = oracle.gae_normalized(ones[:1, :1], ones[:1, :1] * 0, np.zeros((1, 1), np.uint8), gamma=0.9, lam=0.9,
                                      eps=1e-8, ddof=1)
    assert single[0, 0] == 0.0


# ----------------------------------------------------------------------------- Retrace from [N,T,A] tensors
def _probs_case(seed, N=3, T=30, A=4, p=0.08):
    from paper_2608_17641_b200 import workloads
    b = _batch(seed, N=N, T=T, p=p)
    q, pi, mu, act = workloads.make_action_tensors(70, N, T, A, salt=seed)
    return b, q, pi, mu, act


def test_retrace_probs_against_table1_explicit_sum(oracle):
    """alpha_t = r_t + gamma (1 - term_t) E_pi Q(s_{t+1},.) - Q(s_t,a_t), beta_t = gamma c_{t+1} (1 - d_t) with
    c_t = lambda min(c_bar, pi(a_t|s_t)/mu(a_t|s_t)), c_T = 0, carry 0 -- built literally from the tensors."""
    for A in (2, 4, 5):
        b, q, pi, mu, act = _probs_case(40 + A, N=2, T=25, A=A, p=0.1)
        out = oracle.retrace_probs(b["r"], q, pi, mu, act, **_bk(b), gamma=0.99, lam=0.9, c_bar=1.0)
        for n in range(2):
            T = 25
            q64, pi64, mu64 = q[n].astype(float), pi[n].astype(float), mu[n].astype(float)
            eq = (pi64 * q64).sum(axis=1)
            qsa = q64[np.arange(T), act[n]]
            ratio = pi64[np.arange(T), act[n]] / mu64[np.arange(T), act[n]]
            c = float(np.float32(0.9)) * np.minimum(1.0, ratio)
            i = dict(r=b["r"][n], eq=eq, term=b["term"][n], trunc=b["trunc"][n], bv=b["bv"][n], boot=b["boot"][n])
            d = np.maximum(i["term"], i["trunc"]).astype(float)
            alpha = np.array([float(i["r"][t]) + G32 * _table1_successor(eq, i, t, T) - qsa[t] for t in range(T)])
            beta = G32 * np.append(c[1:], 0.0) * (1.0 - d)
            np.testing.assert_allclose(out[n], explicit_sum_backward(alpha, beta, 0.0) + qsa, rtol=1e-12, atol=1e-12)


def test_retrace_probs_reduces_to_scalar_form(oracle):
    """Feeding the scalar-input Retrace with Q(s,a), E_pi Q and log(pi/mu) derived with library routines
    (gather, einsum, log) gives the same targets up to the fp32 rounding of those derived inputs."""
    b, q, pi, mu, act = _probs_case(50, N=4, T=60, A=8)
    out = oracle.retrace_probs(b["r"], q, pi, mu, act, **_bk(b), gamma=0.99, lam=0.95, c_bar=1.5)
    idx = act[..., None].astype(np.int64)
    q_sa = np.take_along_axis(q, idx, axis=2)[..., 0]
    eq = np.einsum("nta,nta->nt", pi.astype(np.float64), q.astype(np.float64)).astype(np.float32)
    lr = np.log(np.take_along_axis(pi, idx, axis=2)[..., 0].astype(np.float64)
                / np.take_along_axis(mu, idx, axis=2)[..., 0].astype(np.float64)).astype(np.float32)
    want = oracle.retrace(b["r"], q_sa, eq, lr, **_bk(b), gamma=0.99, lam=0.95, c_bar=1.5)
    np.testing.assert_allclose(out, want, rtol=2e-5, atol=2e-5)


def test_retrace_probs_structure(oracle):
    b, q, pi, mu, act = _probs_case(51, N=3, T=40, A=4, p=0.0)
    kw = dict(gamma=0.99, lam=0.9, c_bar=1.0)
    base = oracle.retrace_probs(b["r"], q, pi, mu, act, **_bk(b), **kw)
    # relabelling the actions consistently changes nothing
    perm = np.array([2, 0, 3, 1])
    inv = np.argsort(perm)
    out = oracle.retrace_probs(b["r"], q[..., perm], pi[..., perm], mu[..., perm], inv[act].astype(np.int32), **_bk(b), **kw)
    np.testing.assert_allclose(out, base, rtol=1e-13)
    # index shift: the behaviour probabilities of the first step never matter, those of step 5 reach step 4
    mu2 = mu.copy()
    mu2[:, 0, :] = 0.25
    assert np.array_equal(oracle.retrace_probs(b["r"], q, pi, mu2, act, **_bk(b), **kw), base)
    mu3 = mu.copy()
    mu3[:, 5, :] *= 3.0
    out3 = oracle.retrace_probs(b["r"], q, pi, mu3, act, **_bk(b), **kw)
    assert not np.array_equal(out3[:, 4], base[:, 4]) and np.array_equal(out3[:, 5:], base[:, 5:])
    # action-independent Q = V, on-policy, c_bar = 1: target - V = GAE(lambda)
    V = b["V"]
    qv = np.repeat(V[..., None], 4, axis=2)
    on = oracle.retrace_probs(b["r"], qv, pi, pi, act, **_bk(b), gamma=0.99, lam=0.95, c_bar=1.0)
    adv, _ = oracle.gae(b["r"], V, **_bk(b), gamma=0.99, lam=0.95)
    np.testing.assert_allclose(on - V, adv, rtol=1e-6, atol=1e-6)        # sum_a pi = 1 only to fp32 rounding


# ----------------------------------------------------------------------------- vector-valued traces
def test_vector_trace_is_one_scalar_trace_per_component(oracle):
    """Shared scalar decay: component d of the vector trace is the scalar trace of x[:, :, d], exactly."""
    rng = np.random.default_rng(60)
    N, T, D = 3, 50, 6
    x = rng.standard_normal((N, T, D)).astype(np.float32)
    d = (rng.random((N, T)) < 0.1).astype(np.uint8)
    z = oracle.elig_trace_vec(x, d, gamma=0.99, lam=0.9)
    for c in range(D):
        assert np.array_equal(z[:, :, c], oracle.elig_trace(np.ascontiguousarray(x[:, :, c]), d, gamma=0.99, lam=0.9))
    # closed form without flags: z_t = sum_k (gamma lambda)^(t-k) x_k
    z0 = oracle.elig_trace_vec(x, np.zeros((N, T), np.uint8), gamma=0.5, lam=1.0)
    w = 0.5 ** np.arange(T)
    want = np.stack([[np.convolve(x[n, :, c].astype(float), w)[:T] for c in range(D)] for n in range(N)]).transpose(0, 2, 1)
    np.testing.assert_allclose(z0, want, rtol=1e-12, atol=1e-12)


def test_per_dimension_beta_trace_against_the_unrolled_sum(oracle):
    """Eq. 1 unrolled: z_t[c] = sum_k x_k[c] * prod_{s=k+1..t} b_s[c] with b_s = beta_s where the carry into
    s survives and 0 where the flag of step s-1 severs it -- written out with explicit products, no
    recurrence.  Then the special cases: a constant beta reproduces the shared-scalar trace exactly,
    and each component is the generic forward recurrence on its own coefficients."""
    rng = np.random.default_rng(61)
    N, T, D = 2, 12, 3
    x = rng.standard_normal((N, T, D)).astype(np.float32)
    beta = rng.uniform(0.2, 1.1, (N, T, D)).astype(np.float32)
    d = (rng.random((N, T)) < 0.2).astype(np.uint8)
    z = oracle.elig_trace_vec_beta(x, beta, d)
    for n in range(N):
        for c in range(D):
            b = [0.0] + [0.0 if d[n, s - 1] else float(beta[n, s, c]) for s in range(1, T)]
            for t in range(T):
                want = sum(float(x[n, k, c]) * float(np.prod(b[k + 1:t + 1])) for k in range(t + 1))
                assert abs(z[n, t, c] - want) <= 1e-12 * (1 + abs(want)), (n, t, c)
            rec = oracle.linear_recurrence(x[n, :, c].astype(np.float64), np.array(b), 0.0, forward=True)
            np.testing.assert_allclose(z[n, :, c], rec, rtol=1e-13, atol=1e-13)
    const = np.full((N, T, D), 0.25, np.float32)                      # gamma * lambda = 0.5 * 0.5, exact in fp32
    assert np.array_equal(oracle.elig_trace_vec_beta(x, const, d), oracle.elig_trace_vec(x, d, gamma=0.5, lam=0.5))
    # beta at t = 0 is never read
    beta2 = beta.copy()
    beta2[:, 0, :] = np.nan
    assert np.array_equal(oracle.elig_trace_vec_beta(x, beta2, d), z)


# ----------------------------------------------------------------------------- observation-skip masking
def test_skip_masked_gae_is_gae_of_the_sequence_with_masked_steps_deleted(oracle):
    """The reading of Section 9.2's observation-skip masking: masked steps are transparent.  With no
    flag on a masked step, the advantages at the unmasked steps equal plain GAE (an already pinned
    routine) on the row with the masked steps deleted; a masked step repeats the advantage and the
    value of the next unmasked step; the row's trailing masked steps see the window-edge bootstrap."""
    rng = np.random.default_rng(62)
    T = 60
    for trial in range(20):
        r = rng.standard_normal((1, T)).astype(np.float32)
        V = rng.standard_normal((1, T)).astype(np.float32)
        skip = (rng.random((1, T)) < 0.4).astype(np.uint8)
        keep = skip[0] == 0
        if not keep.any():
            continue
        d = ((rng.random((1, T)) < 0.1) & keep).astype(np.uint8)           # flags only on unmasked steps
        tr = ((rng.random((1, T)) < 0.1) & keep).astype(np.uint8)
        bv = rng.standard_normal((1, T)).astype(np.float32)
        boot = rng.standard_normal((1,)).astype(np.float32)
        adv, ret, fil = oracle.gae_skip(r, V, d, tr, bv, boot, skip=skip, gamma=0.97, lam=0.9)
        c = lambda a: np.ascontiguousarray(a[:, keep])
        # the compacted row ends where the original does: trailing masked steps pass the bootstrap through
        want, want_ret = oracle.gae(c(r), c(V), c(d), c(tr), c(bv), boot, gamma=0.97, lam=0.9)
        np.testing.assert_allclose(adv[:, keep], want, rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(ret[:, keep], want_ret, rtol=1e-12, atol=1e-12)
        np.testing.assert_array_equal(fil[:, keep], V[:, keep].astype(np.float64))
        # masked steps repeat what follows them (advantage and value), or the edge values at the end
        for t in range(T - 1, -1, -1):
            if skip[0, t]:
                nxt_a = adv[0, t + 1] if t + 1 < T else 0.0
                nxt_w = fil[0, t + 1] if t + 1 < T else float(boot[0])
                assert adv[0, t] == nxt_a and fil[0, t] == nxt_w and ret[0, t] == nxt_a + nxt_w


def test_skip_masked_gae_special_cases(oracle):
    rng = np.random.default_rng(63)
    N, T = 3, 40
    r, V, bv = (rng.standard_normal((N, T)).astype(np.float32) for _ in range(3))
    d = (rng.random((N, T)) < 0.1).astype(np.uint8)
    tr = (rng.random((N, T)) < 0.1).astype(np.uint8)
    boot = rng.standard_normal((N,)).astype(np.float32)
    # nothing masked: plain GAE, exactly
    adv, ret, fil = oracle.gae_skip(r, V, d, tr, bv, boot, skip=np.zeros((N, T), np.uint8), gamma=0.99, lam=0.95)
    a0, r0 = oracle.gae(r, V, d, tr, bv, boot, gamma=0.99, lam=0.95)
    assert np.array_equal(adv, a0) and np.array_equal(ret, r0) and np.array_equal(fil, V.astype(np.float64))
    # everything masked, no flags: nothing to estimate, the bootstrap shows through every step
    z = np.zeros((N, T), np.uint8)
    adv, ret, fil = oracle.gae_skip(r, V, z, None, None, boot, skip=np.ones((N, T), np.uint8), gamma=0.99, lam=0.95)
    assert not adv.any() and np.array_equal(fil, np.repeat(boot.astype(np.float64)[:, None], T, axis=1))
    # a flagged masked step severs the recurrence: hand-worked row  [u, m(term), u]
    r1 = np.array([[1.0, 5.0, 2.0]], np.float32)
    V1 = np.array([[0.5, 9.0, 0.25]], np.float32)
    d1 = np.array([[0, 1, 0]], np.uint8)
    s1 = np.array([[0, 1, 0]], np.uint8)
    adv, ret, fil = oracle.gae_skip(r1, V1, d1, None, None, np.array([4.0], np.float32), skip=s1, gamma=0.5, lam=0.5)
    # t=2: delta = 2 + 0.5*4 - 0.25 = 3.75 ; t=1 (masked, terminated): A = 0, W = 0 ; t=0: delta = 1 + 0.5*0 - 0.5 = 0.5,
    # continues into the masked step: A = 0.5 + 0.25 * 0 = 0.5
    np.testing.assert_allclose(adv, [[0.5, 0.0, 3.75]], rtol=0, atol=1e-15)
    np.testing.assert_allclose(fil, [[0.5, 0.0, 0.25]], rtol=0, atol=1e-15)
