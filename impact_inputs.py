"""Seeded synthetic inputs for the IMPACT learner hot path.

This module only *draws* inputs: network outputs (logits, means, log-stds, values),
worker actions, rewards and discounts with the shapes of the paper's Atari and MuJoCo
workloads (Section 4.3; hyper-parameter tables of Appendix B).  It holds none of the
loss arithmetic and is the one module that both the CPU oracle's tests and the CUDA
path's tests import.  Everything is NumPy on the host; callers move the arrays where
they need them.

The behaviour (worker) policy's log-probability of the action it took is part of a
worker's sample batch, so it is produced here while sampling the action.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

__all__ = [
    "LossHyper",
    "CONFIGS",
    "categorical_batch",
    "gaussian_batch",
    "round_to_bf16",
    "make_config",
]


@dataclass(frozen=True)
class LossHyper:
    """Scalars of the loss (Algorithm 1; Section 3.1; Appendix B tables)."""

    rho_bar: float = 1.0
    c_bar: float = 1.0
    clip_eps: float = 0.2
    vf_coef: float = 0.5
    ent_coef: float = 0.01
    kl_coef: float = 0.0
    lam: float = 1.0
    rho_tw: float = 1.0
    is_source: int = 0  # 0: target/worker (Section 3.1), 1: learner/worker (Section 2.2), 2: none (rho = c = 1)
    ratio_mode: int = 0  # 0: R3, 1: R1, 2: R2 (Section 4.1)
    objective: int = 0  # 0: epsilon-clipped surrogate (Appendix E), 1: IMPALA's V-trace policy gradient (Section 2.2)


@dataclass(frozen=True)
class Config:
    name: str
    kind: str  # "categorical" | "gaussian"
    B: int
    T: int
    A: int  # actions (categorical) or action dimensions (gaussian)
    seed: int
    p_done: float
    gamma: float
    hyper: LossHyper
    ring_N: int = 0
    ring_K: int = 0
    extra: dict = field(default_factory=dict)


CONFIGS = {
    0: Config("tiny categorical", "categorical", 4, 20, 6, 0, 0.01, 0.99,
              LossHyper(clip_eps=0.2), ring_N=2, ring_K=2),
    1: Config("Atari-shaped categorical", "categorical", 32, 50, 18, 1, 0.01, 0.99,
              LossHyper(clip_eps=0.2), ring_N=16, ring_K=2),
    2: Config("large-batch categorical", "categorical", 1024, 128, 18, 2, 0.005, 0.99,
              LossHyper(clip_eps=0.4), ring_N=32, ring_K=4),
    3: Config("continuous-control Gaussian", "gaussian", 512, 128, 17, 3, 0.001, 0.99,
              LossHyper(clip_eps=0.2, ent_coef=0.0)),
}


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bf16 (ties to even) and return them as fp32.

    Pure bit manipulation, so that the oracle and the CUDA path see the very same
    stored values in the bf16-logits variant.
    """
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    lsb = (u >> np.uint64(16)) & np.uint64(1)
    u = (u + np.uint64(0x7FFF) + lsb) & np.uint64(0xFFFF0000)
    return u.astype(np.uint32).view(np.float32).reshape(x.shape)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """The uint16 storage pattern of values that are already bf16-representable."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    return (x.view(np.uint32) >> np.uint32(16)).astype(np.uint16).reshape(x.shape)


def _log_softmax64(z: np.ndarray) -> np.ndarray:
    z = z.astype(np.float64)
    m = z.max(axis=-1, keepdims=True)
    return z - (m + np.log(np.exp(z - m).sum(axis=-1, keepdims=True)))


def categorical_batch(B: int, T: int, A: int, seed: int, p_done: float = 0.01,
                      gamma: float = 0.99, target_std: float = 0.1,
                      worker_std: float = 0.5, p_reward: float = 0.05) -> dict:
    """One train batch `[B, T]` for a discrete-action policy with `A` actions."""
    rng = np.random.default_rng(seed)
    learner = rng.standard_normal((B, T, A), dtype=np.float32)
    target = (learner + np.float32(target_std) * rng.standard_normal((B, T, A), dtype=np.float32)).astype(np.float32)
    worker = (learner + np.float32(worker_std) * rng.standard_normal((B, T, A), dtype=np.float32)).astype(np.float32)
    lp_w = _log_softmax64(worker)
    # inverse-CDF draw from the worker's softmax
    cdf = np.cumsum(np.exp(lp_w), axis=-1)
    u = rng.random((B, T, 1))
    actions = np.minimum((u > cdf).sum(axis=-1), A - 1).astype(np.int32)
    worker_logp = np.take_along_axis(lp_w, actions[..., None].astype(np.int64), axis=-1)[..., 0].astype(np.float32)
    nonzero = rng.random((B, T)) < p_reward
    sign = np.where(rng.random((B, T)) < 0.5, -1.0, 1.0)
    rewards = (nonzero * sign).astype(np.float32)
    done = rng.random((B, T)) < p_done
    discounts = np.where(done, 0.0, gamma).astype(np.float32)
    values = rng.standard_normal((B, T), dtype=np.float32)
    bootstrap = rng.standard_normal((B,), dtype=np.float32)
    return dict(learner_logits=learner, target_logits=target, worker_logp=worker_logp,
                actions=actions, rewards=rewards, discounts=discounts, values=values,
                bootstrap_values=bootstrap)


def gaussian_batch(B: int, T: int, D: int, seed: int, p_done: float = 0.001,
                   gamma: float = 0.99, target_std: float = 0.05,
                   worker_std: float = 0.3) -> dict:
    """One train batch `[B, T]` for a diagonal-Gaussian policy with `D` action dimensions.

    Only the means of the target and the worker are perturbed; their log-stds equal the
    learner's.
    """
    rng = np.random.default_rng(seed)
    mean = rng.standard_normal((B, T, D), dtype=np.float32)
    logstd = rng.uniform(-1.0, 0.0, (B, T, D)).astype(np.float32)
    t_mean = (mean + np.float32(target_std) * rng.standard_normal((B, T, D), dtype=np.float32)).astype(np.float32)
    w_mean = (mean + np.float32(worker_std) * rng.standard_normal((B, T, D), dtype=np.float32)).astype(np.float32)
    noise = rng.standard_normal((B, T, D))
    sigma = np.exp(logstd.astype(np.float64))
    actions = (w_mean.astype(np.float64) + sigma * noise).astype(np.float32)
    zw = (actions.astype(np.float64) - w_mean.astype(np.float64)) / sigma
    worker_logp = (-0.5 * zw * zw - logstd.astype(np.float64) - 0.5 * np.log(2.0 * np.pi)).sum(axis=-1).astype(np.float32)
    rewards = rng.standard_normal((B, T), dtype=np.float32)
    done = rng.random((B, T)) < p_done
    discounts = np.where(done, 0.0, gamma).astype(np.float32)
    values = rng.standard_normal((B, T), dtype=np.float32)
    bootstrap = rng.standard_normal((B,), dtype=np.float32)
    return dict(learner_mean=mean, learner_logstd=logstd, target_mean=t_mean,
                target_logstd=logstd.copy(), worker_logp=worker_logp, actions=actions,
                rewards=rewards, discounts=discounts, values=values,
                bootstrap_values=bootstrap)


def make_config(idx: int, seed: int | None = None) -> tuple[Config, dict]:
    """Inputs of one of the named configurations (0..3)."""
    cfg = CONFIGS[idx]
    s = cfg.seed if seed is None else seed
    if cfg.kind == "categorical":
        batch = categorical_batch(cfg.B, cfg.T, cfg.A, s, p_done=cfg.p_done, gamma=cfg.gamma)
    else:
        batch = gaussian_batch(cfg.B, cfg.T, cfg.A, s, p_done=cfg.p_done, gamma=cfg.gamma)
    return cfg, batch
