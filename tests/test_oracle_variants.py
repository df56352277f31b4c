"""Pins of the oracle's baseline objectives: PPO's GAE-lambda (Section 2.1) and IMPALA's V-trace policy
gradient (Section 2.2, Appendix D), which reuse the IMPACT recursion with other weights."""
import dataclasses

import numpy as np
import pytest
import torch
from scipy.special import log_softmax

import impact_inputs as ii
from impact_inputs import LossHyper


def _V(b):
    return np.concatenate([b["values"].astype(np.float64), b["bootstrap_values"][:, None].astype(np.float64)], axis=1)


@pytest.mark.parametrize("lam", [0.0, 0.9, 1.0])
def test_no_importance_weights_gives_plain_gae(oracle, lam):
    b = ii.categorical_batch(3, 14, 5, 61, p_done=0.1)
    out = oracle.loss_categorical(b, LossHyper(is_source=2, lam=lam, rho_bar=0.3, c_bar=0.2))
    V, r, g = _V(b), b["rewards"].astype(np.float64), b["discounts"].astype(np.float64)
    td = r + g * V[:, 1:] - V[:, :-1]
    B, T = r.shape
    for bi in range(B):
        for t in range(T):
            # GAE-lambda: sum_i (prod_{j<i} lambda gamma_j) td_i; weights of 1 are above any rho_bar < 1 set here,
            # so truncation must clip them to rho_bar -- unless the source really ignores the policies
            s, coef = 0.0, 1.0
            for i in range(t, T):
                s += coef * min(0.3, 1.0) * td[bi, i]
                coef *= lam * g[bi, i] * min(0.2, 1.0)
            assert out["advantage"][bi, t] == pytest.approx(s, rel=1e-11, abs=1e-13)
    # with the usual bars >= 1 it is textbook GAE: lambda = 0 -> TD error, lambda = 1 -> return - V
    out = oracle.loss_categorical(b, LossHyper(is_source=2, lam=lam))
    if lam == 0.0:
        np.testing.assert_allclose(out["advantage"], td, rtol=1e-12, atol=1e-14)
    if lam == 1.0:
        for bi in range(B):
            for t in range(T):
                ret, coef = 0.0, 1.0
                for i in range(t, T):
                    ret += coef * r[bi, i]
                    coef *= g[bi, i]
                ret += coef * V[bi, T]
                assert out["advantage"][bi, t] == pytest.approx(ret - V[bi, t], rel=1e-10, abs=1e-12)
    # and it does not look at any policy
    b2 = dict(b)
    b2["worker_logp"] = (b["worker_logp"] - 1.0).astype(np.float32)
    out2 = oracle.loss_categorical(b2, LossHyper(is_source=2, lam=lam))
    np.testing.assert_array_equal(out["advantage"], out2["advantage"])


def test_ppo_is_ratio_r2_with_plain_gae(oracle):
    # PPO's objective (Section 2.1): ratio pi_theta / pi_old with pi_old the behaviour policy, GAE advantages
    b = ii.categorical_batch(4, 9, 6, 62)
    h = LossHyper(is_source=2, ratio_mode=2, clip_eps=0.2, lam=0.95, vf_coef=0.0, ent_coef=0.0)
    out = oracle.loss_categorical(b, h)
    lth = np.take_along_axis(log_softmax(b["learner_logits"].astype(np.float64), -1),
                             b["actions"][..., None].astype(np.int64), -1)[..., 0]
    r = np.exp(lth - b["worker_logp"].astype(np.float64))
    adv = out["advantage"]
    L = np.minimum(r * adv, np.clip(r, 0.8, 1.2) * adv).mean()
    assert -out["loss_terms"][1] == pytest.approx(L, rel=1e-12)


def test_vtrace_policy_gradient_weight_and_on_policy_limit(oracle):
    b = ii.categorical_batch(3, 11, 4, 63, p_done=0.1)
    h = LossHyper(objective=1, is_source=1, rho_bar=1.0, c_bar=1.0, lam=1.0, vf_coef=0.0, ent_coef=0.0)
    out = oracle.loss_categorical(b, h)
    lp = log_softmax(b["learner_logits"].astype(np.float64), -1)
    idx = b["actions"][..., None].astype(np.int64)
    lth = np.take_along_axis(lp, idx, -1)[..., 0]
    rho = np.minimum(1.0, np.exp(lth - b["worker_logp"].astype(np.float64)))
    V = _V(b)
    v = np.concatenate([out["vtarget"], b["bootstrap_values"][:, None].astype(np.float64)], axis=1)
    w = rho * (b["rewards"].astype(np.float64) + b["discounts"].astype(np.float64) * v[:, 1:] - V[:, :-1])
    M = w.size
    onehot = np.eye(lp.shape[-1])[b["actions"]]
    np.testing.assert_allclose(out["dlogits"], -(w[..., None]) * (onehot - np.exp(lp)) / M, rtol=1e-11, atol=1e-15)
    assert out["loss_terms"][1] == pytest.approx(-(w * lth).mean(), rel=1e-12)
    assert out["loss_terms"][5] == 0.0  # nothing is clipped in this objective
    np.testing.assert_allclose(out["ratio"], rho, rtol=1e-12)
    # on-policy with lambda = 1: v is the n-step return G, so the weight is r_t + gamma_t G_{t+1} - V_t = G_t - V_t
    bo = dict(b)
    bo["worker_logp"] = lth.astype(np.float32)
    oo = oracle.loss_categorical(bo, h)
    np.testing.assert_allclose(oo["dlogits"] * M, -(oo["advantage"][..., None]) * (onehot - np.exp(lp)), rtol=2e-5, atol=2e-6)


def test_vtrace_policy_gradient_matches_autograd(oracle):
    cfg, b = ii.make_config(0)
    h = dataclasses.replace(cfg.hyper, objective=1, is_source=1, rho_bar=1.2, c_bar=0.9, lam=1.0, kl_coef=0.3)
    out = oracle.loss_categorical(b, h)
    z = torch.tensor(b["learner_logits"], dtype=torch.float64, requires_grad=True)
    pol = torch.distributions.Categorical(logits=z)
    tgt = torch.distributions.Categorical(logits=torch.tensor(b["target_logits"], dtype=torch.float64))
    act = torch.tensor(b["actions"], dtype=torch.int64)
    lth = pol.log_prob(act)
    lw = torch.tensor(b["worker_logp"], dtype=torch.float64)
    values = torch.tensor(b["values"], dtype=torch.float64, requires_grad=True)
    boot = torch.tensor(b["bootstrap_values"], dtype=torch.float64)
    with torch.no_grad():
        wgt = (lth - lw).exp()
        rho, c = wgt.clamp(max=h.rho_bar), wgt.clamp(max=h.c_bar)
        g = torch.tensor(b["discounts"], dtype=torch.float64)
        r = torch.tensor(b["rewards"], dtype=torch.float64)
        vnext = torch.cat([values[:, 1:], boot[:, None]], 1)
        delta = rho * (r + g * vnext - values)
        adv = torch.zeros_like(delta)
        acc = torch.zeros(delta.shape[0], dtype=torch.float64)
        for t in reversed(range(delta.shape[1])):
            acc = delta[:, t] + h.lam * g[:, t] * c[:, t] * acc
            adv[:, t] = acc
        vt = values + adv
        vt_next = torch.cat([vt[:, 1:], boot[:, None]], 1)
        w = rho * (r + g * vt_next - values)
    total = (-(w * lth).mean() + h.vf_coef * (0.5 * (values - vt) ** 2).mean() - h.ent_coef * pol.entropy().mean()
             + h.kl_coef * torch.distributions.kl_divergence(tgt, pol).mean())
    dz, dv = torch.autograd.grad(total, [z, values])
    assert out["loss_terms"][0] == pytest.approx(total.item(), rel=1e-12)
    np.testing.assert_allclose(out["dlogits"], dz.numpy(), rtol=1e-9, atol=1e-15)
    np.testing.assert_allclose(out["dvalues"], dv.numpy(), rtol=1e-9, atol=1e-15)


def test_gaussian_variants_share_the_recursion(oracle):
    b = ii.gaussian_batch(3, 8, 4, 64, p_done=0.1)
    base = LossHyper(ent_coef=0.0, lam=0.9)
    gae = oracle.loss_gaussian(b, dataclasses.replace(base, is_source=2))
    V, r, g = _V(b), b["rewards"].astype(np.float64), b["discounts"].astype(np.float64)
    td = r + g * V[:, 1:] - V[:, :-1]
    acc = np.zeros(r.shape[0])
    for t in reversed(range(r.shape[1])):
        acc = td[:, t] + 0.9 * g[:, t] * acc
        np.testing.assert_allclose(gae["advantage"][:, t], acc, rtol=1e-12, atol=1e-14)
    pg = oracle.loss_gaussian(b, dataclasses.replace(base, objective=1, is_source=1, vf_coef=0.0))
    assert pg["loss_terms"][5] == 0.0 and np.isfinite(pg["dmean"]).all()
