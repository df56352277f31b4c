"""The workspace-free loss call for embedders that may not allocate device memory.

`impact_loss_fwd_bwd_static_scratch` serves hosts such as a plugin running inside another
framework's memory pool, or a control loop that must never block in the driver's allocator:
its scratch is an array inside the library, so the caller passes inputs and outputs only.
The check here is that it returns what the ordinary call returns, twice in a row (the
second call starts from whatever the first left in the shared array), that both agree with
the CPU oracle, that every kernel behind the entry point (persistent, tile-sweeping,
runtime-width; fp32 and bf16 storage) is reached through it, and that it refuses batches
the array is too small for.  The file name keeps it last in collection order.
"""
import numpy as np
import pytest
import torch

import impact_inputs as ii

pytestmark = pytest.mark.gpu


def _device_batch(idx):
    cfg, batch = ii.make_config(idx)
    return cfg, {k: torch.from_numpy(v).cuda() for k, v in batch.items()}


def _outputs(B, T, A):
    return dict(loss_terms=torch.full((8,), float("nan"), device="cuda"),
                dlogits=torch.full((B, T, A), float("nan"), device="cuda"),
                dvalues=torch.full((B, T), float("nan"), device="cuda"),
                vtarget=torch.full((B, T), float("nan"), device="cuda"),
                advantage=torch.full((B, T), float("nan"), device="cuda"))


def _args(t):
    return (t["learner_logits"], t["target_logits"], t["worker_logp"], t["actions"], t["rewards"],
            t["discounts"], t["values"], t["bootstrap_values"])


@pytest.mark.parametrize("idx", [1, 2])
def test_static_scratch_call_matches_the_workspace_call_twice_in_a_row(idx, oracle):
    import paper_1912_00167_b200 as ip
    import _parity as P
    cfg, t = _device_batch(idx)
    B, T, A = cfg.B, cfg.T, cfg.A
    h = cfg.hyper
    coef = ip.Coefficients(rho_bar=h.rho_bar, c_bar=h.c_bar, clip_eps=h.clip_eps, vf_coef=h.vf_coef,
                           ent_coef=h.ent_coef, kl_coef=0.25, lam=0.995, rho_tw=2.0)
    want = _outputs(B, T, A)
    ip.impact_loss_fwd_bwd(*_args(t), coef, workspace=ip.new_workspace(B, T), **want)
    torch.cuda.synchronize()
    M = B * T
    for attempt in range(2):
        got = _outputs(B, T, A)
        ip.impact_loss_fwd_bwd_static_scratch(*_args(t), coef, **got)
        torch.cuda.synchronize()
        for key in ("dlogits", "dvalues"):  # gradients carry 1/M: compare on their natural scale
            np.testing.assert_allclose(got[key].cpu().numpy() * M, want[key].cpu().numpy() * M,
                                       rtol=1e-5, atol=1e-6, err_msg=f"{key}, call {attempt}")
        for key in ("vtarget", "advantage"):
            np.testing.assert_allclose(got[key].cpu().numpy(), want[key].cpu().numpy(), rtol=1e-5, atol=1e-6,
                                       err_msg=f"{key}, call {attempt}")
        np.testing.assert_allclose(got["loss_terms"].cpu().numpy(), want["loss_terms"].cpu().numpy(),
                                   rtol=1e-4, atol=1e-7, err_msg=f"loss_terms, call {attempt}")
    assert ip.impact_loss_static_scratch_status() == 0
    # and against the oracle itself, on the bar of the other parity tests
    import dataclasses
    h2 = P.f32_hyper(dataclasses.replace(h, kl_coef=0.25, lam=0.995, rho_tw=2.0))
    batch = ii.make_config(idx)[1]
    ref = oracle.loss_categorical(batch, h2)
    near = P.near_clip_bound(ref, h2)
    flipped = oracle.loss_categorical(batch, h2, flip=near.astype(np.int8)) if near.any() else None
    sens = P._policy_sensitivity(oracle.loss_categorical, batch, h2, ["dlogits"], M,
                                 near.astype(np.int8) if near.any() else None)
    gpu = {k: v.float().cpu().numpy().astype(np.float64) for k, v in got.items()}
    P.compare(gpu, ref, flipped, near, M, ["dlogits"], h2.kl_coef, sens, h2.vf_coef)


@pytest.mark.parametrize("B,T,A,dtype", [(5, 300, 18, torch.float32), (3, 200, 64, torch.float32),
                                         (9, 50, 18, torch.bfloat16), (4, 40, 33, torch.float32),
                                         (301, 21, 9, torch.bfloat16)])
def test_static_scratch_call_reaches_every_kernel(B, T, A, dtype):
    """Long trajectories (swept tile by tile inside a block, partial sums and ticket in the built-in array), wide
    rows without room for tile aggregates (runtime-width kernel), bf16 storage, an action count with no compiled
    kernel, tiles that start inside a 16-byte granule: each against the workspace call, twice."""
    import paper_1912_00167_b200 as ip
    batch = ii.categorical_batch(B, T, A, seed=77 + B + T + A, p_done=0.02)
    t = {k: torch.from_numpy(v).cuda() for k, v in batch.items()}
    t["learner_logits"], t["target_logits"] = t["learner_logits"].to(dtype), t["target_logits"].to(dtype)
    coef = ip.Coefficients(rho_bar=1.2, c_bar=1.0, clip_eps=0.3, kl_coef=0.1, lam=0.97, rho_tw=2.0)

    def outputs():
        o = _outputs(B, T, A)
        o["dlogits"] = o["dlogits"].to(dtype)
        return o
    want = outputs()
    ip.impact_loss_fwd_bwd(*_args(t), coef, workspace=ip.new_workspace(1, 1), **want)  # fixed part only: no aggregates
    torch.cuda.synchronize()
    for attempt in range(2):
        got = outputs()
        ip.impact_loss_fwd_bwd_static_scratch(*_args(t), coef, **got)
        torch.cuda.synchronize()
        for key in want:
            assert torch.equal(got[key], want[key]), f"{key}, call {attempt}"  # same kernel, same order of sums
    assert ip.impact_loss_static_scratch_status() == 0


def test_static_scratch_call_refuses_what_does_not_fit():
    import paper_1912_00167_b200 as ip
    from paper_1912_00167_b200 import binding as bd
    # 1025 trajectories of 128 steps: one tile more than the built-in scratch holds
    B, T, A = 1025, 128, 6
    t = {k: torch.from_numpy(v).cuda() for k, v in ii.categorical_batch(B, T, A, seed=5).items()}
    out = _outputs(B, T, A)
    with pytest.raises(ip.ImpactError) as e:
        ip.impact_loss_fwd_bwd_static_scratch(*_args(t), ip.Coefficients(), **out)
    assert e.value.status == bd.ERR_WORKSPACE_TOO_SMALL
    assert torch.isnan(out["loss_terms"]).all()  # nothing was enqueued
    # rows of 64 actions are worked on in tiles of 64 steps: 1025 such tiles do not fit either
    B, T, A = 1025, 64, 64
    t = {k: torch.from_numpy(v).cuda() for k, v in ii.categorical_batch(B, T, A, seed=7).items()}
    with pytest.raises(ip.ImpactError) as e:
        ip.impact_loss_fwd_bwd_static_scratch(*_args(t), ip.Coefficients(), **_outputs(B, T, A))
    assert e.value.status == bd.ERR_WORKSPACE_TOO_SMALL
    # too many actions for this variant
    B, T, A = 4, 8, 65
    t = {k: torch.from_numpy(v).cuda() for k, v in ii.categorical_batch(B, T, A, seed=6).items()}
    with pytest.raises(ip.ImpactError) as e:
        ip.impact_loss_fwd_bwd_static_scratch(*_args(t), ip.Coefficients(), **_outputs(B, T, A))
    assert e.value.status == bd.ERR_UNSUPPORTED
    # and a batch that fits still runs afterwards
    cfg, t = _device_batch(0)
    out = _outputs(cfg.B, cfg.T, cfg.A)
    ip.impact_loss_fwd_bwd_static_scratch(*_args(t), ip.Coefficients(), **out)
    torch.cuda.synchronize()
    assert torch.isfinite(out["loss_terms"]).all()
