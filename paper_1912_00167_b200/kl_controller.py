"""Caller-side controller of the KL coefficient eta of Algorithm 1.

The paper's hyper-parameter tables carry a "KL Target" next to the initial "KL Coeff" but never state how
eta follows it.  This helper applies the rule PPO was published with (Schulman et al. 2017, "Proximal Policy
Optimization Algorithms", Section 4, adaptive KL penalty): after a policy update, with d the measured mean
KL(pi_target || pi_theta) -- `loss_terms[IMPACT_TERM_KL]` of the loss call --

    d < d_target / 1.5  ->  eta <- eta / 2
    d > d_target * 1.5  ->  eta <- eta * 2

and eta unchanged in between.  It is host logic only: the next loss call gets `kl_coef = controller.eta`.
(The loss call evaluates the KL term only while kl_coef != 0, so eta never reaches 0 here.)
"""
from __future__ import annotations

from dataclasses import dataclass


@dataclass
class AdaptiveKL:
    eta: float = 1.0          # current coefficient (the tables' "KL Coeff" to start with)
    kl_target: float = 0.01   # the tables' "KL Target"
    band: float = 1.5         # tolerance factor around the target
    factor: float = 2.0       # multiplicative step
    eta_min: float = 1e-8
    eta_max: float = 1e8

    def __post_init__(self):
        if not (self.eta > 0 and self.kl_target > 0 and self.band >= 1 and self.factor > 1):
            raise ValueError("need eta > 0, kl_target > 0, band >= 1, factor > 1")

    def update(self, measured_kl: float) -> float:
        """Adjusts and returns eta given the mean KL of the batch just trained on."""
        if measured_kl != measured_kl:  # NaN: leave eta alone
            return self.eta
        if measured_kl < self.kl_target / self.band:
            self.eta = max(self.eta / self.factor, self.eta_min)
        elif measured_kl > self.kl_target * self.band:
            self.eta = min(self.eta * self.factor, self.eta_max)
        return self.eta
