"""Pins of the CPU oracle's loss against what the paper and the mathematics fix.

Nothing here calls the CUDA path.  Every expected value is computed by a route that
differs from the oracle's own (double loops over the defining sums, closed forms,
probability-space instead of log-space, finite differences, autograd on library ops).
"""
import dataclasses

import numpy as np
import pytest
import torch
from scipy.special import log_softmax

import impact_inputs as ii
from impact_inputs import LossHyper


def _cat(B, T, A, seed, **kw):
    return ii.categorical_batch(B, T, A, seed, **kw)


def _lp_taken(z, a):
    lp = log_softmax(z.astype(np.float64), axis=-1)
    return np.take_along_axis(lp, a[..., None].astype(np.int64), axis=-1)[..., 0]


def _on_policy(batch):
    """All three policies coincide: target = learner, worker log-prob = learner log-prob."""
    b = dict(batch)
    b["target_logits"] = b["learner_logits"].copy()
    b["worker_logp"] = _lp_taken(b["learner_logits"], b["actions"]).astype(np.float32)
    return b


# --- Section 2.2 / 3.1: on-policy reduction to n-step returns ---------------------------
@pytest.mark.parametrize("rho_bar,c_bar", [(1.0, 1.0), (3.0, 1.5)])
def test_on_policy_vtrace_is_discounted_n_step_return(oracle, rho_bar, c_bar):
    b = _on_policy(_cat(5, 17, 6, 11, p_done=0.1))
    h = LossHyper(rho_bar=rho_bar, c_bar=c_bar, lam=1.0)
    out = oracle.loss_categorical(b, h)
    B, T = b["rewards"].shape
    # worker_logp is the fp32 rounding of the learner's log-prob, so the ratio is 1 to ~1e-7
    for bi in range(B):
        for t in range(T):
            g, ret = 1.0, 0.0
            for i in range(t, T):
                ret += g * float(b["rewards"][bi, i])
                g *= float(b["discounts"][bi, i])
            ret += g * float(b["bootstrap_values"][bi])
            assert out["vtarget"][bi, t] == pytest.approx(ret, rel=2e-6, abs=2e-6)


def test_on_policy_gradient_is_advantage_weighted_logprob_gradient(oracle):
    b = _on_policy(_cat(3, 9, 5, 12))
    h = LossHyper(rho_bar=1.0, c_bar=1.0, clip_eps=0.2, vf_coef=0.0, ent_coef=0.0, rho_tw=1.0)
    out = oracle.loss_categorical(b, h)
    M = b["rewards"].size
    pi = np.exp(log_softmax(b["learner_logits"].astype(np.float64), axis=-1))
    onehot = np.eye(pi.shape[-1])[b["actions"]]
    expect = -(out["advantage"][..., None]) * (onehot - pi) / M
    np.testing.assert_allclose(out["dlogits"], expect, rtol=1e-6, atol=1e-9)
    np.testing.assert_allclose(out["ratio"], 1.0, rtol=1e-6)


# --- Section 2.2 and 3.1: the defining sums, evaluated literally ------------------------
@pytest.mark.parametrize("lam", [1.0, 0.995])
@pytest.mark.parametrize("is_source", [0, 1])
def test_advantage_equals_brute_force_sum(oracle, lam, is_source):
    rng = np.random.default_rng(5)
    b = _cat(3, 12, 4, 21, p_done=0.0)
    gamma = float(np.float32(0.97))  # the discount as stored
    b["discounts"][:] = gamma
    rho_bar, c_bar = float(rng.uniform(0.5, 2.0)), float(rng.uniform(0.5, 2.0))
    h = LossHyper(rho_bar=rho_bar, c_bar=c_bar, lam=lam, is_source=is_source)
    out = oracle.loss_categorical(b, h)
    lt = _lp_taken(b["target_logits"], b["actions"])
    lth = _lp_taken(b["learner_logits"], b["actions"])
    w = np.exp((lth if is_source else lt) - b["worker_logp"].astype(np.float64))
    rho, c = np.minimum(rho_bar, w), np.minimum(c_bar, w)
    B, T = w.shape
    V = np.concatenate([b["values"].astype(np.float64), b["bootstrap_values"][:, None].astype(np.float64)], axis=1)
    r = b["rewards"].astype(np.float64)
    for bi in range(B):
        for t in range(T):
            s = 0.0
            for i in range(t, T):
                prod_c = 1.0
                for j in range(t, i):
                    prod_c *= c[bi, j]
                td = rho[bi, i] * (r[bi, i] + gamma * V[bi, i + 1] - V[bi, i])
                s += (lam * gamma) ** (i - t) * prod_c * td
            assert out["advantage"][bi, t] == pytest.approx(s, rel=1e-11, abs=1e-12)
            assert out["vtarget"][bi, t] == pytest.approx(V[bi, t] + s, rel=1e-11, abs=1e-12)


def test_per_step_discounts_replace_powers_of_gamma(oracle):
    b = _cat(2, 10, 4, 22, p_done=0.3)
    h = LossHyper(rho_bar=1.3, c_bar=0.9, lam=0.9)
    out = oracle.loss_categorical(b, h)
    lt = _lp_taken(b["target_logits"], b["actions"])
    w = np.exp(lt - b["worker_logp"].astype(np.float64))
    rho, c = np.minimum(1.3, w), np.minimum(0.9, w)
    g = b["discounts"].astype(np.float64)
    V = np.concatenate([b["values"].astype(np.float64), b["bootstrap_values"][:, None].astype(np.float64)], axis=1)
    B, T = w.shape
    for bi in range(B):
        for t in range(T):
            s = 0.0
            for i in range(t, T):
                coef = 1.0
                for j in range(t, i):
                    coef *= 0.9 * g[bi, j] * c[bi, j]
                s += coef * rho[bi, i] * (float(b["rewards"][bi, i]) + g[bi, i] * V[bi, i + 1] - V[bi, i])
            assert out["advantage"][bi, t] == pytest.approx(s, rel=1e-11, abs=1e-12)


def test_closed_form_constant_reward(oracle):
    T, gamma, vT = 25, 0.9, 0.7
    b = _on_policy(_cat(2, T, 3, 23))
    b["rewards"][:] = 1.0
    b["values"][:] = 0.0
    b["discounts"][:] = gamma
    b["bootstrap_values"][:] = vT
    out = oracle.loss_categorical(b, LossHyper())
    g32 = float(np.float32(gamma))
    v32 = float(np.float32(vT))
    for t in range(T):
        n = T - t
        expect = (1 - g32 ** n) / (1 - g32) + g32 ** n * v32
        np.testing.assert_allclose(out["vtarget"][:, t], expect, rtol=3e-6)


# --- truncation of the importance weights (Section 2.2) ----------------------------------
def test_truncation_and_one_step_limit(oracle):
    b = _cat(4, 15, 6, 24)
    lt = _lp_taken(b["target_logits"], b["actions"])
    w = np.exp(lt - b["worker_logp"].astype(np.float64))
    assert (w > 1.0).any() and (w < 1.0).any()
    V = np.concatenate([b["values"].astype(np.float64), b["bootstrap_values"][:, None].astype(np.float64)], axis=1)
    td = b["rewards"].astype(np.float64) + b["discounts"].astype(np.float64) * V[:, 1:] - V[:, :-1]
    # c_bar = 0: the trace is cut everywhere, the advantage is rho_t times the 1-step TD error
    for rho_bar in (0.7, 1.0, 1e30):
        out = oracle.loss_categorical(b, LossHyper(rho_bar=rho_bar, c_bar=0.0))
        np.testing.assert_allclose(out["advantage"], np.minimum(rho_bar, w) * td, rtol=1e-12, atol=1e-14)
        assert out["loss_terms"][6] == pytest.approx((w > rho_bar).mean())
    # the weight never exceeds rho_bar: |A_t| <= rho_bar |td|
    out = oracle.loss_categorical(b, LossHyper(rho_bar=0.7, c_bar=0.0))
    assert (np.abs(out["advantage"]) <= 0.7 * np.abs(td) + 1e-14).all()


def test_episode_end_cuts_bootstrap_and_trace(oracle):
    b = _cat(2, 12, 4, 25, p_done=0.0)
    cut = 6
    b["discounts"][:, cut] = 0.0
    h = LossHyper(rho_bar=1.5, c_bar=1.2, lam=0.95)
    out = oracle.loss_categorical(b, h)
    lt = _lp_taken(b["target_logits"], b["actions"])
    rho = np.minimum(1.5, np.exp(lt - b["worker_logp"].astype(np.float64)))
    expect = rho[:, cut] * (b["rewards"][:, cut].astype(np.float64) - b["values"][:, cut].astype(np.float64))
    np.testing.assert_allclose(out["advantage"][:, cut], expect, rtol=1e-12)
    # nothing after the cut reaches the steps up to it
    b2 = {k: v.copy() for k, v in b.items()}
    b2["rewards"][:, cut + 1:] += 3.0
    b2["values"][:, cut + 1:] -= 2.0
    b2["bootstrap_values"][:] = 9.0
    out2 = oracle.loss_categorical(b2, h)
    np.testing.assert_array_equal(out["advantage"][:, :cut + 1], out2["advantage"][:, :cut + 1])
    assert not np.allclose(out["advantage"][:, cut + 1:], out2["advantage"][:, cut + 1:])


# --- Section 3.1 / Algorithm 1: the ratio and its gradient -------------------------------
def test_huge_clip_eps_gives_algorithm_1_gradient(oracle):
    b = _cat(3, 8, 5, 26)
    rho_tw = 2.0
    h = LossHyper(rho_bar=1.0, c_bar=1.0, clip_eps=1e9, vf_coef=0.0, ent_coef=0.0, rho_tw=rho_tw)
    out = oracle.loss_categorical(b, h)
    M = b["rewards"].size
    p_th = np.exp(log_softmax(b["learner_logits"].astype(np.float64), axis=-1))
    p_tg = np.exp(log_softmax(b["target_logits"].astype(np.float64), axis=-1))
    idx = b["actions"][..., None].astype(np.int64)
    pth_a = np.take_along_axis(p_th, idx, -1)[..., 0]
    ptg_a = np.take_along_axis(p_tg, idx, -1)[..., 0]
    pw_a = np.exp(b["worker_logp"].astype(np.float64))
    # grad pi_theta(a) wrt logits = pi_theta(a) (onehot - pi_theta), divided by max(pi_target, beta pi_worker)
    onehot = np.eye(p_th.shape[-1])[b["actions"]]
    grad_J = (pth_a / np.maximum(ptg_a, pw_a / rho_tw) * out["advantage"])[..., None] * (onehot - p_th) / M
    np.testing.assert_allclose(out["dlogits"], -grad_J, rtol=1e-10, atol=1e-14)
    assert out["loss_terms"][5] == 0.0


@pytest.mark.parametrize("rho_tw", [1.0, 2.0, 5.0])
def test_min_form_equals_max_form(oracle, rho_tw):
    # Section 3.1: min(pi_w/pi_t, rho) pi_theta/pi_w  ==  pi_theta / max(pi_t, pi_w / rho)
    b = _cat(4, 10, 6, 27, worker_std=1.5)
    out = oracle.loss_categorical(b, LossHyper(rho_tw=rho_tw))
    idx = b["actions"][..., None].astype(np.int64)
    pth = np.take_along_axis(np.exp(log_softmax(b["learner_logits"].astype(np.float64), -1)), idx, -1)[..., 0]
    ptg = np.take_along_axis(np.exp(log_softmax(b["target_logits"].astype(np.float64), -1)), idx, -1)[..., 0]
    pw = np.exp(b["worker_logp"].astype(np.float64))
    min_form = np.minimum(pw / ptg, rho_tw) * pth / pw
    np.testing.assert_allclose(out["ratio"], min_form, rtol=1e-12)
    assert ((pw / ptg) > rho_tw).any() and ((pw / ptg) < rho_tw).any()


@pytest.mark.parametrize("mode,den", [(1, "target"), (2, "worker")])
def test_ablation_ratios(oracle, mode, den):
    b = _cat(3, 7, 5, 28)
    out = oracle.loss_categorical(b, LossHyper(ratio_mode=mode, rho_tw=2.0))
    lth = _lp_taken(b["learner_logits"], b["actions"])
    d = _lp_taken(b["target_logits"], b["actions"]) if den == "target" else b["worker_logp"].astype(np.float64)
    np.testing.assert_allclose(out["ratio"], np.exp(lth - d), rtol=1e-12)


def _single_step(oracle, l_th, l_tg, l_w, adv, eps, rho_tw=1.0, ratio_mode=0):
    """One step, two actions; log-probs of action 0 are set through the logits."""
    def logits(lp0):
        p0 = np.exp(lp0)
        return np.array([[[np.log(p0), np.log1p(-p0)]]], dtype=np.float64)
    zl, zt = logits(l_th), logits(l_tg)
    b = dict(learner_logits=zl.astype(np.float32), target_logits=zt.astype(np.float32),
             worker_logp=np.array([[l_w]], np.float32), actions=np.zeros((1, 1), np.int32),
             rewards=np.array([[adv]], np.float32), discounts=np.zeros((1, 1), np.float32),
             values=np.zeros((1, 1), np.float32), bootstrap_values=np.zeros((1,), np.float32))
    # rho_bar huge, discount 0, value 0: advantage = rho * reward; use rho_bar to keep rho = its raw value
    h = LossHyper(rho_bar=1e30, c_bar=1.0, clip_eps=eps, vf_coef=0.0, ent_coef=0.0, rho_tw=rho_tw,
                  ratio_mode=ratio_mode)
    out = oracle.loss_categorical(b, h)
    return out


def test_gradient_vanishes_beyond_clip_bounds(oracle):
    eps = 0.2
    l_tg = np.log(0.4)
    l_w = np.log(0.3)  # worker below target: denominator is the target's probability
    for R, sign, clipped in [(1.5, +1, True), (1.5, -1, False), (0.5, -1, True), (0.5, +1, False),
                             (1.1, +1, False), (0.9, -1, False)]:
        l_th = l_tg + np.log(R)
        out = _single_step(oracle, l_th, l_tg, l_w, sign * 1.0, eps)
        assert out["ratio"][0, 0] == pytest.approx(R, rel=1e-6)
        adv = out["advantage"][0, 0]
        assert np.sign(adv) == sign
        s = -out["loss_terms"][1]
        if clipped:
            assert np.all(out["dlogits"] == 0.0)
            assert s == pytest.approx((1 + eps if R > 1 else 1 - eps) * adv, rel=1e-6)
            assert out["loss_terms"][5] == 1.0
        else:
            assert np.all(out["dlogits"] != 0.0)
            assert s == pytest.approx(R * adv, rel=1e-6)
            assert out["loss_terms"][5] == 0.0
    # continuity of the surrogate across the bound
    s_in = -_single_step(oracle, l_tg + np.log(1.2 - 1e-6), l_tg, l_w, 1.0, eps)["loss_terms"][1]
    s_out = -_single_step(oracle, l_tg + np.log(1.2 + 1e-6), l_tg, l_w, 1.0, eps)["loss_terms"][1]
    assert abs(s_in - s_out) < 1e-5


def test_impact_clip_is_lower_bound_of_ppo_clip(oracle):
    # Appendix E: with rho = 1 and a non-negative advantage, the IMPACT target eps-clip
    # objective lies below PPO's eps-clip objective (ratio pi_theta / pi_worker).
    rng = np.random.default_rng(3)
    for _ in range(200):
        l_th, l_tg, l_w = np.log(rng.uniform(0.05, 0.9, 3))
        adv = float(rng.uniform(0.1, 2.0))
        eps = float(rng.uniform(0.1, 0.4))
        s_impact = -_single_step(oracle, l_th, l_tg, l_w, adv, eps, rho_tw=1.0, ratio_mode=0)["loss_terms"][1]
        s_ppo = -_single_step(oracle, l_th, l_tg, l_w, adv, eps, ratio_mode=2)["loss_terms"][1]
        assert s_impact <= s_ppo + 1e-9


# --- Algorithm 1: gradients against finite differences with frozen targets ---------------
def _total_frozen_categorical(z, values, b, adv, vtarget, h):
    lp = log_softmax(z, axis=-1)
    idx = b["actions"][..., None].astype(np.int64)
    lth = np.take_along_axis(lp, idx, -1)[..., 0]
    lpt = log_softmax(b["target_logits"].astype(np.float64), axis=-1)
    ltg = np.take_along_axis(lpt, idx, -1)[..., 0]
    lw = b["worker_logp"].astype(np.float64)
    d = np.maximum(ltg, lw - np.log(h.rho_tw))
    R = np.exp(lth - d)
    surr = np.minimum(R * adv, np.clip(R, 1 - h.clip_eps, 1 + h.clip_eps) * adv)
    ent = -(np.exp(lp) * lp).sum(-1)
    kl = (np.exp(lpt) * (lpt - lp)).sum(-1)
    return (-surr.mean() + h.vf_coef * (0.5 * (values - vtarget) ** 2).mean()
            - h.ent_coef * ent.mean() + h.kl_coef * kl.mean())


def test_categorical_gradients_match_finite_differences(oracle):
    cfg, b = ii.make_config(0)
    h = dataclasses.replace(cfg.hyper, kl_coef=0.3, rho_tw=2.0, lam=0.995, rho_bar=1.2)
    out = oracle.loss_categorical(b, h)
    z0 = b["learner_logits"].astype(np.float64)
    v0 = b["values"].astype(np.float64)
    f0 = _total_frozen_categorical(z0, v0, b, out["advantage"], out["vtarget"], h)
    assert f0 == pytest.approx(out["loss_terms"][0], rel=1e-12)
    hstep = 1e-6
    # steps whose ratio sits within the FD step of a clip bound are skipped (kink)
    R = out["ratio"]
    smooth = (np.abs(R - (1 + h.clip_eps)) > 1e-4) & (np.abs(R - (1 - h.clip_eps)) > 1e-4)
    B, T, A = z0.shape
    for bi in range(B):
        for t in range(T):
            if not smooth[bi, t]:
                continue
            for k in range(A):
                zp, zm = z0.copy(), z0.copy()
                zp[bi, t, k] += hstep
                zm[bi, t, k] -= hstep
                fd = (_total_frozen_categorical(zp, v0, b, out["advantage"], out["vtarget"], h)
                      - _total_frozen_categorical(zm, v0, b, out["advantage"], out["vtarget"], h)) / (2 * hstep)
                assert out["dlogits"][bi, t, k] == pytest.approx(fd, rel=2e-5, abs=2e-9)
            vp, vm = v0.copy(), v0.copy()
            vp[bi, t] += hstep
            vm[bi, t] -= hstep
            fd = (_total_frozen_categorical(z0, vp, b, out["advantage"], out["vtarget"], h)
                  - _total_frozen_categorical(z0, vm, b, out["advantage"], out["vtarget"], h)) / (2 * hstep)
            assert out["dvalues"][bi, t] == pytest.approx(fd, rel=2e-5, abs=2e-9)


def test_dlogits_rows_sum_to_zero(oracle):
    cfg, b = ii.make_config(1)
    h = dataclasses.replace(cfg.hyper, kl_coef=0.5, rho_tw=2.0)
    out = oracle.loss_categorical(b, h)
    scale = np.abs(out["dlogits"]).sum(-1)
    assert (np.abs(out["dlogits"].sum(-1)) <= 1e-13 * (1 + scale)).all()


def test_entropy_and_kl_special_cases(oracle):
    b = _cat(3, 6, 7, 29)
    b["learner_logits"][:] = 0.37
    h = LossHyper(ent_coef=1.0, vf_coef=0.0, clip_eps=0.0)
    # clip_eps = 0 and R != 1: whether the policy term passes does not matter below, only entropy
    out = oracle.loss_categorical(b, h)
    assert out["loss_terms"][3] == pytest.approx(np.log(7.0), rel=1e-12)
    b2 = _on_policy(_cat(3, 6, 7, 30))
    out2 = oracle.loss_categorical(b2, LossHyper(kl_coef=1.0, ent_coef=0.0, vf_coef=0.0))
    assert abs(out2["loss_terms"][4]) < 1e-15
    # uniform policy: entropy term contributes no gradient; on-policy: KL contributes none
    out3 = oracle.loss_categorical(b2, LossHyper(kl_coef=0.0, ent_coef=0.0, vf_coef=0.0))
    np.testing.assert_allclose(out2["dlogits"], out3["dlogits"], atol=1e-16)
    b["target_logits"][:] = b["learner_logits"]
    b["worker_logp"][:] = np.float32(-np.log(7.0))
    o_ent = oracle.loss_categorical(b, LossHyper(ent_coef=1.0, vf_coef=0.0))
    o_no = oracle.loss_categorical(b, LossHyper(ent_coef=0.0, vf_coef=0.0))
    np.testing.assert_allclose(o_ent["dlogits"], o_no["dlogits"], atol=1e-15)


def test_total_combines_terms(oracle):
    cfg, b = ii.make_config(0)
    h = dataclasses.replace(cfg.hyper, kl_coef=0.7, vf_coef=0.3, ent_coef=0.05)
    lt = oracle.loss_categorical(b, h)["loss_terms"]
    assert lt[0] == pytest.approx(lt[1] + 0.3 * lt[2] - 0.05 * lt[3] + 0.7 * lt[4], rel=1e-14)
    assert lt[3] > 0 and lt[4] > 0 and lt[2] > 0


# --- second opinion: autograd over library ops -------------------------------------------
def _torch_total(b, h, gaussian=False):
    t64 = lambda x: torch.tensor(np.asarray(x), dtype=torch.float64)
    lw = t64(b["worker_logp"])
    if gaussian:
        mu = t64(b["learner_mean"]).requires_grad_()
        ls = t64(b["learner_logstd"]).requires_grad_()
        pol = torch.distributions.Normal(mu, ls.exp())
        tgt = torch.distributions.Normal(t64(b["target_mean"]), t64(b["target_logstd"]).exp())
        act = t64(b["actions"])
        lth, ltg = pol.log_prob(act).sum(-1), tgt.log_prob(act).sum(-1)
        ent = pol.entropy().sum(-1)
        kl = torch.distributions.kl_divergence(tgt, pol).sum(-1)
        leaves = [mu, ls]
    else:
        z = t64(b["learner_logits"]).requires_grad_()
        pol = torch.distributions.Categorical(logits=z)
        tgt = torch.distributions.Categorical(logits=t64(b["target_logits"]))
        act = torch.tensor(b["actions"], dtype=torch.int64)
        lth, ltg = pol.log_prob(act), tgt.log_prob(act)
        ent = pol.entropy()
        kl = torch.distributions.kl_divergence(tgt, pol)
        leaves = [z]
    values = t64(b["values"]).requires_grad_()
    leaves.append(values)
    with torch.no_grad():
        x = (lth if h.is_source == 1 else ltg) - lw
        rho = x.exp().clamp(max=h.rho_bar)
        c = x.exp().clamp(max=h.c_bar)
        g = t64(b["discounts"])
        vnext = torch.cat([values[:, 1:], t64(b["bootstrap_values"])[:, None]], dim=1)
        delta = rho * (t64(b["rewards"]) + g * vnext - values)
        adv = torch.zeros_like(delta)
        acc = torch.zeros(delta.shape[0], dtype=torch.float64)
        for t in reversed(range(delta.shape[1])):
            acc = delta[:, t] + h.lam * g[:, t] * c[:, t] * acc
            adv[:, t] = acc
        vtarget = values + adv
    d = torch.maximum(ltg, lw - np.log(h.rho_tw)).detach()
    R = (lth - d).exp()
    surr = torch.minimum(R * adv, R.clamp(1 - h.clip_eps, 1 + h.clip_eps) * adv)
    total = (-surr.mean() + h.vf_coef * (0.5 * (values - vtarget) ** 2).mean()
             - h.ent_coef * ent.mean() + h.kl_coef * kl.mean())
    grads = torch.autograd.grad(total, leaves)
    return total.item(), [g_.numpy() for g_ in grads], adv.numpy(), vtarget.numpy()


@pytest.mark.parametrize("idx,is_source", [(0, 0), (1, 0), (1, 1)])
def test_categorical_matches_autograd(oracle, idx, is_source):
    cfg, b = ii.make_config(idx)
    h = dataclasses.replace(cfg.hyper, kl_coef=0.25, rho_tw=2.0, lam=0.995, rho_bar=1.1, c_bar=0.9,
                            is_source=is_source)
    out = oracle.loss_categorical(b, h)
    total, (dz, dv), adv, vt = _torch_total(b, h)
    assert out["loss_terms"][0] == pytest.approx(total, rel=1e-12)
    np.testing.assert_allclose(out["advantage"], adv, rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(out["dlogits"], dz, rtol=1e-9, atol=1e-15)
    np.testing.assert_allclose(out["dvalues"], dv, rtol=1e-9, atol=1e-15)


def test_gaussian_matches_autograd(oracle):
    b = ii.gaussian_batch(6, 11, 5, 31, p_done=0.05)
    b["target_logstd"] = (b["target_logstd"] + 0.1 * np.random.default_rng(1).standard_normal(b["target_logstd"].shape)).astype(np.float32)
    h = LossHyper(rho_bar=1.1, c_bar=0.9, clip_eps=0.3, vf_coef=0.5, ent_coef=0.02, kl_coef=0.4,
                  lam=0.995, rho_tw=2.0)
    out = oracle.loss_gaussian(b, h)
    total, (dmu, dls, dv), adv, vt = _torch_total(b, h, gaussian=True)
    assert out["loss_terms"][0] == pytest.approx(total, rel=1e-12)
    np.testing.assert_allclose(out["advantage"], adv, rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(out["dmean"], dmu, rtol=1e-9, atol=1e-15)
    np.testing.assert_allclose(out["dlogstd"], dls, rtol=1e-9, atol=1e-15)
    np.testing.assert_allclose(out["dvalues"], dv, rtol=1e-9, atol=1e-15)


# --- Gaussian closed forms ---------------------------------------------------------------
def test_gaussian_closed_forms(oracle):
    B, T, D = 2, 5, 4
    b = ii.gaussian_batch(B, T, D, 32)
    for k in ("learner_logstd", "target_logstd"):
        b[k][:] = 0.0
    b["target_mean"] = b["learner_mean"].copy()
    b["actions"] = b["learner_mean"].copy()  # a = mu, sigma = 1
    lp = -0.5 * D * np.log(2 * np.pi)
    b["worker_logp"][:] = np.float32(lp)
    h = LossHyper(ent_coef=0.5, kl_coef=1.0, vf_coef=0.0, rho_bar=10.0)
    out = oracle.loss_gaussian(b, h)
    assert out["loss_terms"][3] == pytest.approx(0.5 * D * np.log(2 * np.pi * np.e), rel=1e-12)
    assert abs(out["loss_terms"][4]) < 1e-15
    np.testing.assert_allclose(out["ratio"], 1.0, rtol=1e-6)  # fp32 rounding of worker_logp only
    # at a = mu: d log pi / d mu = 0, d log pi / d logstd = -1
    M = B * T
    np.testing.assert_allclose(out["dmean"], 0.0, atol=1e-18)
    w = out["advantage"] * out["ratio"] * (1.0 - 0.0)
    clipped = np.zeros_like(w)  # R = 1 is inside the interval
    expect = (-(w)[..., None] * (-1.0) - 0.5) / M * np.ones((B, T, D))
    np.testing.assert_allclose(out["dlogstd"], expect, rtol=1e-12)


def test_gaussian_gradients_match_finite_differences(oracle):
    b = ii.gaussian_batch(2, 6, 3, 33, p_done=0.0)
    h = LossHyper(rho_bar=1.2, c_bar=1.0, clip_eps=0.3, vf_coef=0.5, ent_coef=0.03, kl_coef=0.2, rho_tw=2.0)
    out = oracle.loss_gaussian(b, h)
    adv, vt = out["advantage"], out["vtarget"]

    def total(mu, ls, values):
        a = b["actions"].astype(np.float64)
        mut, lst = b["target_mean"].astype(np.float64), b["target_logstd"].astype(np.float64)
        c0 = 0.5 * np.log(2 * np.pi)
        lth = (-0.5 * ((a - mu) / np.exp(ls)) ** 2 - ls - c0).sum(-1)
        ltg = (-0.5 * ((a - mut) / np.exp(lst)) ** 2 - lst - c0).sum(-1)
        d = np.maximum(ltg, b["worker_logp"].astype(np.float64) - np.log(h.rho_tw))
        R = np.exp(lth - d)
        surr = np.minimum(R * adv, np.clip(R, 1 - h.clip_eps, 1 + h.clip_eps) * adv)
        ent = (ls + c0 + 0.5).sum(-1)
        kl = (ls - lst + (np.exp(2 * lst) + (mut - mu) ** 2) / (2 * np.exp(2 * ls)) - 0.5).sum(-1)
        return (-surr.mean() + h.vf_coef * (0.5 * (values - vt) ** 2).mean()
                - h.ent_coef * ent.mean() + h.kl_coef * kl.mean())

    mu0, ls0, v0 = (b[k].astype(np.float64) for k in ("learner_mean", "learner_logstd", "values"))
    assert total(mu0, ls0, v0) == pytest.approx(out["loss_terms"][0], rel=1e-12)
    R = out["ratio"]
    smooth = (np.abs(R - 1.3) > 1e-4) & (np.abs(R - 0.7) > 1e-4)
    eps = 1e-6
    for idx in np.ndindex(mu0.shape):
        if not smooth[idx[:2]]:
            continue
        for name, base, grad in (("mu", mu0, out["dmean"]), ("ls", ls0, out["dlogstd"])):
            p, m = base.copy(), base.copy()
            p[idx] += eps
            m[idx] -= eps
            if name == "mu":
                fd = (total(p, ls0, v0) - total(m, ls0, v0)) / (2 * eps)
            else:
                fd = (total(mu0, p, v0) - total(mu0, m, v0)) / (2 * eps)
            assert grad[idx] == pytest.approx(fd, rel=5e-5, abs=5e-9)


def test_bf16_rounding_helper_is_round_to_nearest_even():
    x = np.array([1.0, 1.00390625, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, -2.71828, 3.0e-5], np.float32)
    r = ii.round_to_bf16(x)
    expect = torch.tensor(x).to(torch.bfloat16).to(torch.float32).numpy()
    np.testing.assert_array_equal(r, expect)
    big = np.random.default_rng(0).standard_normal(10000).astype(np.float32)
    np.testing.assert_array_equal(ii.round_to_bf16(big), torch.tensor(big).to(torch.bfloat16).float().numpy())


def test_the_two_test_hooks_of_the_oracle_are_what_the_tests_take_them_for(oracle):
    """`adv_cond` and `flip` are not part of the loss; the GPU parity tests take their tolerance and their "other
    valid branch" from them, so both are pinned here against evaluations that do not go through the oracle's
    recursion: adv_cond against the defining double sum over |terms|, flip against the difference it must make
    (the policy term of exactly the marked steps, present in one run and absent in the other)."""
    cfg, batch = ii.make_config(0)
    h = dataclasses.replace(cfg.hyper, lam=0.97, rho_bar=1.3, c_bar=1.1, clip_eps=0.25, kl_coef=0.0)
    ref = oracle.loss_categorical(batch, h)
    B, T = batch["rewards"].shape
    lp_t = log_softmax(batch["target_logits"].astype(np.float64), axis=-1)
    l_t = np.take_along_axis(lp_t, batch["actions"][..., None], -1)[..., 0]
    w = np.exp(l_t - batch["worker_logp"].astype(np.float64))
    rho, c = np.minimum(w, h.rho_bar), np.minimum(w, h.c_bar)
    r, g, v = (batch[k].astype(np.float64) for k in ("rewards", "discounts", "values"))
    v_next = np.concatenate([v[:, 1:], batch["bootstrap_values"].astype(np.float64)[:, None]], 1)
    term = rho * (np.abs(r) + np.abs(g * v_next) + np.abs(v))
    want = np.zeros((B, T))
    for b in range(B):
        for t in range(T):
            prod = 1.0
            for i in range(t, T):  # sum_i |prod_{j<i} lambda gamma_j c_j| * |terms of delta_i|
                want[b, t] += prod * term[b, i]
                prod *= abs(h.lam * g[b, i] * c[b, i])
    np.testing.assert_allclose(ref["adv_cond"], want, rtol=1e-12, atol=0)
    assert (ref["adv_cond"] >= np.abs(ref["advantage"]) * (1 - 1e-12)).all()

    flip = np.zeros((B, T), np.int8)
    flip[1, 3] = flip[2, 7] = 1
    other = oracle.loss_categorical(batch, h, flip=flip)
    changed = np.abs(other["dlogits"] - ref["dlogits"]).max(-1) > 0
    assert (changed == (flip == 1)).all()
    for key in ("advantage", "vtarget", "dvalues", "ratio"):
        np.testing.assert_array_equal(other[key], ref[key])
    # the difference is the policy term of the marked steps: -A R (onehot - pi) / M, present on one side only
    pi = np.exp(log_softmax(batch["learner_logits"].astype(np.float64), axis=-1))
    onehot = np.eye(pi.shape[-1])[batch["actions"]]
    term_pg = -(ref["advantage"] * ref["ratio"])[..., None] * (onehot - pi) / (B * T)
    for (b, t) in ((1, 3), (2, 7)):
        diff = other["dlogits"][b, t] - ref["dlogits"][b, t]
        assert np.allclose(diff, term_pg[b, t], rtol=1e-10, atol=1e-18) or np.allclose(diff, -term_pg[b, t], rtol=1e-10, atol=1e-18)
