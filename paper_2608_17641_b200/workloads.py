"""Seeded synthetic rollout tensors (numpy, host side).

This module draws inputs only -- it holds none of the method's arithmetic -- so
that the CUDA path and the CPU oracle can be fed the very same arrays.  Every
tensor gets its own generator stream: seed = 17641000 + 100*config + tensor_id.

The shapes and distributions are those of the five benchmark configurations
(random tensors of the paper's rollout regimes: 8x128 "standard PPO",
4096 x {32..1024} massively parallel simulation, 64x16384 RLHF-length rows,
16384x2048 bandwidth-saturating batch); the paper's own workloads are random
tensors of these shapes as well, there is no dataset behind them.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

_TENSOR_IDS = {
    "rewards": 1, "values": 2, "q_sa": 3, "expected_q": 4, "log_rhos": 5, "dones": 6, "truncs": 7,
    "trunc_bootstrap": 8, "bootstrap": 9, "x": 10,
}


def _rng(config: int, name: str, salt: int = 0) -> np.random.Generator:
    return np.random.default_rng(17641 * 1000 + 100 * config + _TENSOR_IDS[name] + 100000 * salt)


def _normal(config, name, shape, scale=1.0, salt=0):
    out = _rng(config, name, salt).standard_normal(shape, dtype=np.float32)
    if scale != 1.0:
        out *= np.float32(scale)
    return out


def _bernoulli(config, name, shape, p, salt=0):
    return (_rng(config, name, salt).random(shape, dtype=np.float32) < np.float32(p)).astype(np.uint8)


@dataclass
class Rollout:
    """One batch of synthetic rollout tensors; every [N,T] array is C-contiguous."""
    N: int
    T: int
    rewards: np.ndarray
    values: np.ndarray
    dones: np.ndarray                     # d^term, uint8
    bootstrap: np.ndarray                 # [N] window-edge value
    truncs: np.ndarray | None = None      # d^trunc, uint8
    trunc_bootstrap: np.ndarray | None = None   # [N,T] continuation values at truncations
    q_sa: np.ndarray | None = None
    expected_q: np.ndarray | None = None
    log_rhos: np.ndarray | None = None
    x: np.ndarray | None = None
    params: dict = field(default_factory=dict)

    @property
    def any_done(self) -> np.ndarray:
        """term OR trunc: the single flag the two forward scans take."""
        if self.truncs is None:
            return self.dones
        return ((self.dones != 0) | (self.truncs != 0)).astype(np.uint8)


def make_rollout(config: int, N: int, T: int, *, p_done=0.02, p_trunc=0.005, with_truncs=True,
                 all_algorithms=True, gamma=0.99, lam=0.95, salt=0) -> Rollout:
    """Dense-reward rollout: r, V (and q, E_pi q, x) ~ N(0,1); log pi - log mu ~ N(0, 0.5^2);
    dones ~ Bernoulli(p_done); truncs ~ Bernoulli(p_trunc); both bootstraps ~ N(0,1)."""
    shape = (N, T)
    ro = Rollout(
        N=N, T=T,
        rewards=_normal(config, "rewards", shape, salt=salt),
        values=_normal(config, "values", shape, salt=salt),
        dones=_bernoulli(config, "dones", shape, p_done, salt=salt),
        bootstrap=_normal(config, "bootstrap", (N,), salt=salt),
        params=dict(gamma=gamma, lam=lam, rho_bar=1.0, c_bar=1.0),
    )
    if with_truncs:
        ro.truncs = _bernoulli(config, "truncs", shape, p_trunc, salt=salt)
        ro.trunc_bootstrap = _normal(config, "trunc_bootstrap", shape, salt=salt)
    if all_algorithms:
        ro.q_sa = _normal(config, "q_sa", shape, salt=salt)
        ro.expected_q = _normal(config, "expected_q", shape, salt=salt)
        ro.log_rhos = _normal(config, "log_rhos", shape, scale=0.5, salt=salt)
        ro.x = _normal(config, "x", shape, salt=salt)
    return ro


def config1(salt=0) -> Rollout:
    """GAE 8x128, dones 1%, truncs 0.5%, gamma .99, lambda .95."""
    return make_rollout(1, 8, 128, p_done=0.01, p_trunc=0.005, all_algorithms=False, salt=salt)


def config2(salt=0) -> Rollout:
    """All seven algorithms, 4096x64, dones 2%, truncs 0.5%."""
    return make_rollout(2, 4096, 64, salt=salt)


def config3(T: int, with_truncs: bool, N: int = 4096, salt=0) -> Rollout:
    """GAE / V-Trace sweep member: 4096 x T, with or without per-step truncation handling."""
    return make_rollout(3, N, T, with_truncs=with_truncs, salt=salt)


def config4(N: int = 64, T: int = 16384, salt=0) -> Rollout:
    """Long-row RLHF-like batch: gamma = 1, dones 0.1%, no truncations; the reward is zero except
    ~N(0,1) at the last step of each segment (every done step and t = T-1)."""
    shape = (N, T)
    dones = _bernoulli(4, "dones", shape, 1e-3, salt=salt)
    seg_end = dones.astype(bool).copy()
    seg_end[:, -1] = True
    rewards = np.where(seg_end, _normal(4, "rewards", shape, salt=salt), np.float32(0.0)).astype(np.float32)
    return Rollout(
        N=N, T=T, rewards=rewards, values=_normal(4, "values", shape, salt=salt), dones=dones,
        bootstrap=_normal(4, "bootstrap", (N,), salt=salt),
        params=dict(gamma=1.0, lam=0.95, rho_bar=1.0, c_bar=1.0),
    )


def config5(N: int = 16384, T: int = 2048, salt=0) -> Rollout:
    """Bandwidth-saturating batch: all seven algorithms, truncation handling on."""
    return make_rollout(5, N, T, salt=salt)


def make_action_tensors(config: int, N: int, T: int, A: int, salt=0):
    """[N,T,A] Q-values ~ N(0,1), target / behaviour action probabilities (softmax of N(0,1) logits; the
    behaviour logits are the target logits plus N(0, 0.5^2) noise, so log pi - log mu has the spread
    of the scalar-input configurations) and int32 actions [N,T] drawn from the behaviour policy."""
    rng = np.random.default_rng(17641 * 1000 + 100 * config + 50 + 100000 * salt + 7 * A)
    q = rng.standard_normal((N, T, A), dtype=np.float32)
    logits = rng.standard_normal((N, T, A), dtype=np.float32)
    blogits = logits + np.float32(0.5) * rng.standard_normal((N, T, A), dtype=np.float32)

    def softmax(z):
        z = z - z.max(axis=2, keepdims=True)
        e = np.exp(z, dtype=np.float32)
        return (e / e.sum(axis=2, keepdims=True)).astype(np.float32)

    pi, mu = softmax(logits), softmax(blogits)
    u = rng.random((N, T, 1), dtype=np.float32)
    actions = np.minimum((np.cumsum(mu, axis=2) < u).sum(axis=2), A - 1).astype(np.int32)
    return q, pi, mu, actions
