"""Parity of the CUDA loss kernels with the CPU oracle, element by element, through the C ABI."""
import dataclasses

import numpy as np
import pytest
import torch

import impact_inputs as ii
from impact_inputs import LossHyper

import _parity as P

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("idx", [0, 1, 2])
def test_named_categorical_configs(oracle, idx):
    cfg, batch = ii.make_config(idx)
    P.check_categorical(oracle, batch, cfg.hyper)


@pytest.mark.parametrize("idx", [0, 1, 2])
def test_named_configs_with_paper_hyperparameters(oracle, idx):
    # Appendix B: rho = 2, lambda = 0.995, plus a KL term
    cfg, batch = ii.make_config(idx)
    h = dataclasses.replace(cfg.hyper, rho_tw=2.0, lam=0.995, kl_coef=0.5, vf_coef=1.0, clip_eps=0.3)
    P.check_categorical(oracle, batch, h)


def test_config2_bf16_logits(oracle):
    cfg, batch = ii.make_config(2)
    P.check_categorical(oracle, batch, cfg.hyper, torch.bfloat16, torch.bfloat16,
                        rtol=P.RTOL_BF16, atol=P.ATOL_BF16)
    # bf16 storage with fp32 gradients: only the inputs are rounded, so the fp32 bar holds
    P.check_categorical(oracle, batch, cfg.hyper, torch.bfloat16, torch.float32)
    P.check_categorical(oracle, batch, cfg.hyper, torch.float32, torch.bfloat16,
                        rtol=P.RTOL_BF16, atol=P.ATOL_BF16)


def test_config3_gaussian(oracle):
    cfg, batch = ii.make_config(3)
    P.check_gaussian(oracle, batch, cfg.hyper)
    h = dataclasses.replace(cfg.hyper, rho_tw=2.0, lam=0.995, kl_coef=1.0, ent_coef=0.01, clip_eps=0.4,
                            rho_bar=1.5, c_bar=1.2)
    P.check_gaussian(oracle, batch, h)


SHAPES = [
    (1, 1, 1), (1, 1, 7), (3, 1, 4), (1, 5, 2), (7, 33, 3), (5, 127, 6), (4, 128, 18), (3, 129, 18),
    (2, 300, 5), (9, 50, 18), (2, 20, 65), (3, 40, 64), (2, 70, 100), (1, 9, 257), (2, 5, 512),
    (130, 1, 18), (65, 2, 9), (3, 1000, 4),
]


@pytest.mark.parametrize("B,T,A", SHAPES)
def test_ragged_shapes_categorical(oracle, B, T, A):
    batch = ii.categorical_batch(B, T, A, seed=1000 + B * 7 + T * 3 + A, p_done=0.05)
    h = LossHyper(rho_bar=1.3, c_bar=1.1, clip_eps=0.25, vf_coef=0.7, ent_coef=0.02, kl_coef=0.1,
                  lam=0.97, rho_tw=2.0)
    P.check_categorical(oracle, batch, h)


@pytest.mark.parametrize("B,T,D", [(1, 1, 1), (3, 7, 3), (5, 128, 17), (2, 131, 6), (4, 50, 33), (1, 300, 64),
                                   (2, 9, 256), (40, 3, 17)])
def test_ragged_shapes_gaussian(oracle, B, T, D):
    batch = ii.gaussian_batch(B, T, D, seed=2000 + B + T + D, p_done=0.02)
    h = LossHyper(rho_bar=1.3, c_bar=1.1, clip_eps=0.25, vf_coef=0.7, ent_coef=0.02, kl_coef=0.1,
                  lam=0.97, rho_tw=2.0)
    P.check_gaussian(oracle, batch, h)


@pytest.mark.parametrize("B,T,A", [(3, 33, 5), (6, 20, 18), (2, 129, 7), (5, 50, 64)])
def test_bf16_ragged(oracle, B, T, A):
    batch = ii.categorical_batch(B, T, A, seed=3000 + A, p_done=0.05)
    h = LossHyper(rho_tw=2.0, kl_coef=0.2, lam=0.995)
    P.check_categorical(oracle, batch, h, torch.bfloat16, torch.bfloat16, rtol=P.RTOL_BF16, atol=P.ATOL_BF16)
    P.check_categorical(oracle, batch, h, torch.bfloat16, torch.float32)


@pytest.mark.parametrize("B,T,A,dtype", [(301, 21, 9, torch.bfloat16), (77, 21, 6, torch.bfloat16),
                                         (50, 25, 9, torch.float32), (1311, 50, 18, torch.bfloat16),
                                         (2000, 21, 9, torch.bfloat16), (151, 127, 18, torch.bfloat16)])
def test_tiles_that_start_and_end_inside_a_16_byte_granule(oracle, B, T, A, dtype):
    """Row pitches that are no multiple of 16 bytes: every tile (or the last one) starts or ends inside a granule, so
    the bulk copies are widened to the enclosing granules, the ends of the gradient rows and of the copied target
    rows leave byte by byte, and the tensors' last partial granule comes by ordinary loads.  Few tiles per block
    and more tiles than stages; the target logits are copied out as on a batch's first traversal."""
    batch = ii.categorical_batch(B, T, A, seed=4100 + B + T + A, p_done=0.02)
    plain = LossHyper(rho_bar=1.0, c_bar=1.0, clip_eps=0.3, vf_coef=0.5, ent_coef=0.01, kl_coef=0.0, rho_tw=1.0)
    full = LossHyper(rho_bar=1.3, c_bar=1.1, clip_eps=0.25, vf_coef=0.7, ent_coef=0.02, kl_coef=0.1, lam=0.97, rho_tw=2.0)
    if dtype == torch.bfloat16:
        P.check_categorical(oracle, batch, plain, dtype, dtype, extra=False, target_copy=True, rtol=P.RTOL_BF16,
                            atol=P.ATOL_BF16)
        P.check_categorical(oracle, batch, full, dtype, torch.float32, target_copy=True)
        P.check_categorical(oracle, batch, plain, torch.float32, dtype, extra=False, target_copy=True, rtol=P.RTOL_BF16,
                            atol=P.ATOL_BF16)
    else:
        P.check_categorical(oracle, batch, plain, extra=False, target_copy=True)
        P.check_categorical(oracle, batch, full, target_copy=True)


@pytest.mark.parametrize("idx", [0, 1, 2])
def test_named_configs_compare_the_kl_term_too(oracle, idx):
    """The named configurations have kl_coef = 0, where the library does not evaluate the KL term (and reports 0,
    which the other tests assert).  With a coefficient of 1e-20 the term is evaluated and weighs nothing: every
    output including mean KL is compared with the oracle."""
    cfg, batch = ii.make_config(idx)
    P.check_categorical(oracle, batch, dataclasses.replace(cfg.hyper, kl_coef=1e-20))


def test_nan_and_inf_inputs_propagate_and_nothing_hangs():
    """No input is sanitised: a NaN logit or an infinite reward shows up in the outputs that depend on it (and in
    the batch means), the gradients of the trajectories in other tiles are those of the clean batch, and no wait
    gives up.  (Short trajectories share a 128-step tile, and the recursion's cut between them is a multiplication
    by zero, which a non-finite value survives: it may also reach the trajectories before it in its own tile.)"""
    import paper_1912_00167_b200 as ip
    cfg, batch = ii.make_config(1)
    B, T, A = cfg.B, cfg.T, cfg.A
    clean = {k: torch.from_numpy(v).cuda() for k, v in batch.items()}
    dirty = {k: v.clone() for k, v in clean.items()}
    dirty["learner_logits"][3, 10, 2] = float("nan")
    dirty["rewards"][7, 20] = float("inf")
    dirty["target_logits"][9, 0, 0] = float("-inf")  # a target probability of exactly 0: legal
    coef = P.to_coef(P.f32_hyper(cfg.hyper))
    res = []
    for t in (clean, dirty):
        out = dict(loss_terms=torch.zeros(8, device="cuda"), dlogits=torch.zeros(B, T, A, device="cuda"),
                   dvalues=torch.zeros(B, T, device="cuda"), advantage=torch.zeros(B, T, device="cuda"))
        ws = ip.new_workspace(B, T)
        ip.impact_loss_fwd_bwd(t["learner_logits"], t["target_logits"], t["worker_logp"], t["actions"], t["rewards"],
                               t["discounts"], t["values"], t["bootstrap_values"], coef, workspace=ws, **out)
        torch.cuda.synchronize()
        assert ip.impact_loss_workspace_status(ws) == 0
        res.append(out)
    c, d = res
    assert torch.isfinite(c["dlogits"]).all() and torch.isfinite(c["loss_terms"]).all()
    assert torch.isnan(d["dlogits"][3, 10]).all()           # the row with the NaN logit
    assert not torch.isfinite(d["advantage"][7, 20])        # the step with the infinite reward ...
    assert not torch.isfinite(d["advantage"][7, :21]).any() or cfg.hyper.c_bar == 0  # ... and the steps before it
    assert not torch.isfinite(d["loss_terms"][0])           # the batch means carry it
    per_tile = 128 // T
    hit = {b_ // per_tile for b_ in (3, 7)}
    untouched = [b for b in range(B) if b // per_tile not in hit and b != 9]
    assert torch.equal(d["dlogits"][untouched], c["dlogits"][untouched])
    assert torch.equal(d["dvalues"][untouched], c["dvalues"][untouched])
    assert torch.isfinite(d["dlogits"][9]).all()            # -inf target logit: probability 0, finite everything


def test_out_of_range_actions_are_clamped():
    """Actions outside [0, A) are clamped into range by the kernels (the oracle refuses them): the outputs are
    those of the batch with the clamped actions, bit for bit."""
    import paper_1912_00167_b200 as ip
    for (B, T, A) in ((6, 40, 18), (5, 30, 33), (4, 200, 6)):
        batch = ii.categorical_batch(B, T, A, seed=31 + A)
        t = {k: torch.from_numpy(v).cuda() for k, v in batch.items()}
        bad = t["actions"].clone()
        bad[0, 0], bad[1, 5], bad[2, T - 1] = -3, A, A + 1000
        outs = []
        for act in (bad, bad.clamp(0, A - 1)):
            out = dict(loss_terms=torch.zeros(8, device="cuda"), dlogits=torch.zeros(B, T, A, device="cuda"),
                       dvalues=torch.zeros(B, T, device="cuda"))
            ip.impact_loss_fwd_bwd(t["learner_logits"], t["target_logits"], t["worker_logp"], act, t["rewards"],
                                   t["discounts"], t["values"], t["bootstrap_values"], ip.Coefficients(kl_coef=0.1),
                                   workspace=ip.new_workspace(B, T), **out)
            torch.cuda.synchronize()
            outs.append(out)
        for k in outs[0]:
            assert torch.equal(outs[0][k], outs[1][k]), k


@pytest.mark.parametrize("B,T,A", [(300, 64, 64), (7, 128, 64), (3, 200, 64), (1500, 20, 64), (33, 63, 64)])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_wide_rows_in_the_persistent_kernel(oracle, B, T, A, dtype):
    """A = 64: tiles of 64 steps, rows streamed from shared memory with a skewed walk; one tile per trajectory,
    several trajectories per tile, trajectories over two and four tiles, more tiles per block than stages; the
    default configuration (switches compiled out) and the full one."""
    batch = ii.categorical_batch(B, T, A, seed=640 + B + T, p_done=0.01)
    plain = LossHyper(rho_bar=1.0, c_bar=1.0, clip_eps=0.3, vf_coef=0.5, ent_coef=0.01, kl_coef=0.0, rho_tw=1.0)
    full = LossHyper(rho_bar=1.3, c_bar=1.1, clip_eps=0.25, vf_coef=0.7, ent_coef=0.02, kl_coef=0.1, lam=0.97, rho_tw=2.0)
    if dtype == torch.bfloat16:
        P.check_categorical(oracle, batch, plain, torch.bfloat16, torch.bfloat16, extra=False, rtol=P.RTOL_BF16,
                            atol=P.ATOL_BF16)
        P.check_categorical(oracle, batch, full, torch.bfloat16, torch.float32)
    else:
        P.check_categorical(oracle, batch, plain, extra=False)
        P.check_categorical(oracle, batch, full)


@pytest.mark.parametrize("B,T,A,dtype", [(2, 4500, 6, torch.float32), (5, 1300, 9, torch.float32),
                                         (1, 130, 18, torch.float32), (40, 257, 18, torch.bfloat16),
                                         (700, 256, 18, torch.float32), (3, 640, 4, torch.float32)])
def test_long_trajectories_split_across_blocks(oracle, B, T, A, dtype):
    """T > 128: the tiles of a trajectory are worked on by different blocks at once and linked through their
    published aggregates (more than 32 tiles per trajectory, a partial first tile, rows that end unaligned);
    from a few hundred trajectories on a block sweeps a trajectory by itself."""
    batch = ii.categorical_batch(B, T, A, seed=900 + B + T + A, p_done=0.003)
    h = LossHyper(rho_bar=1.2, c_bar=1.0, clip_eps=0.3, vf_coef=0.5, ent_coef=0.01, kl_coef=0.05, lam=0.99, rho_tw=2.0)
    if dtype == torch.bfloat16:
        P.check_categorical(oracle, batch, h, torch.bfloat16, torch.float32)
    else:
        P.check_categorical(oracle, batch, h)
    P.check_categorical(oracle, batch, dataclasses.replace(h, objective=1, kl_coef=0.0), dtype, torch.float32)


@pytest.mark.parametrize("B,T,D", [(2, 4500, 3), (5, 1024, 17), (1, 130, 6), (30, 300, 17), (500, 256, 6)])
def test_gaussian_long_trajectories(oracle, B, T, D):
    """T > 128 for the compiled action dimensions: tiles of a trajectory on different blocks, linked through their
    aggregates (few trajectories), or swept inside one block (many)."""
    batch = ii.gaussian_batch(B, T, D, seed=7000 + B + T + D, p_done=0.003)
    P.check_gaussian(oracle, batch, LossHyper(rho_bar=1.2, c_bar=1.0, clip_eps=0.3, vf_coef=0.5, ent_coef=0.01,
                                              kl_coef=0.05, lam=0.99, rho_tw=2.0))
    P.check_gaussian(oracle, batch, LossHyper(objective=1))


@pytest.mark.parametrize("B,T,D", [(41, 21, 17), (301, 50, 6), (1500, 128, 6), (900, 128, 3), (700, 100, 17),
                                   (149, 128, 17), (33, 127, 3)])
def test_gaussian_persistent_kernel_shapes(oracle, B, T, D):
    """The compiled action dimensions with T <= 128: several trajectories per tile, tiles that end
    unaligned, a ragged last tile, one tile more than there are SMs, and more tiles per block than the
    ring has stages; with and without the KL term."""
    batch = ii.gaussian_batch(B, T, D, seed=5000 + B + T + D, p_done=0.01)
    P.check_gaussian(oracle, batch, LossHyper(rho_bar=1.0, c_bar=1.0, clip_eps=0.3, vf_coef=0.5, ent_coef=0.01,
                                              kl_coef=0.0, rho_tw=1.0))
    if B < 400:
        P.check_gaussian(oracle, batch, LossHyper(rho_bar=1.3, c_bar=1.1, clip_eps=0.25, vf_coef=0.7, ent_coef=0.02,
                                                  kl_coef=0.1, lam=0.97, rho_tw=2.0))


@pytest.mark.parametrize("mode", [1, 2])
@pytest.mark.parametrize("is_source", [0, 1])
def test_variants(oracle, mode, is_source):
    cfg, batch = ii.make_config(1)
    h = dataclasses.replace(cfg.hyper, ratio_mode=mode, is_source=is_source, rho_tw=2.0)
    P.check_categorical(oracle, batch, h)


def test_degenerate_coefficients(oracle):
    cfg, batch = ii.make_config(1)
    for h in (LossHyper(c_bar=0.0), LossHyper(rho_bar=0.0), LossHyper(clip_eps=0.0, ent_coef=0.0),
              LossHyper(vf_coef=0.0, ent_coef=0.0, kl_coef=0.0, lam=0.0)):
        P.check_categorical(oracle, batch, h)
    # no truncation at all: |lambda gamma c| exceeds 1 on many steps, the recursion amplifies
    # rounding, and fewer elements stay inside the purely relative bar (the conditioned one holds)
    P.check_categorical(oracle, batch, LossHyper(rho_bar=float("inf"), c_bar=float("inf"), clip_eps=1e9),
                        min_literal=0.98)


def test_all_steps_terminal_and_on_policy(oracle):
    batch = ii.categorical_batch(6, 40, 8, seed=77)
    batch["discounts"][:] = 0.0
    P.check_categorical(oracle, batch, LossHyper())
    batch = ii.categorical_batch(6, 40, 8, seed=78)
    batch["target_logits"] = batch["learner_logits"].copy()
    P.check_categorical(oracle, batch, LossHyper(kl_coef=1.0))


@pytest.mark.parametrize("B,T,A", [(4, 20, 6), (32, 50, 18), (1024, 128, 18), (7, 33, 4), (5, 127, 9), (130, 1, 18),
                                   (301, 21, 9), (1500, 128, 6), (2000, 50, 18)])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_default_configuration_without_optional_outputs(oracle, B, T, A, dtype):
    """No KL term, default ratio and importance weights, no vtarget / advantage: the configuration for which the
    library compiles its switches out.  Shapes cover one and several trajectories per tile, tiles that end
    unaligned, a ragged last tile, and more tiles per block than the ring has stages."""
    batch = ii.categorical_batch(B, T, A, seed=31 + B + T + A, p_done=0.02)
    h = LossHyper(rho_bar=1.0, c_bar=1.0, clip_eps=0.3, vf_coef=0.5, ent_coef=0.01, kl_coef=0.0, rho_tw=1.0)
    if dtype == torch.bfloat16:
        P.check_categorical(oracle, batch, h, torch.bfloat16, torch.bfloat16, extra=False, rtol=P.RTOL_BF16,
                            atol=P.ATOL_BF16)
    else:
        P.check_categorical(oracle, batch, h, extra=False)


def test_optional_outputs_can_be_skipped_and_results_are_deterministic(oracle):
    cfg, batch = ii.make_config(1)
    h = P.f32_hyper(cfg.hyper)
    a = P.run_gpu_categorical(batch, h, extra=True)
    b = P.run_gpu_categorical(batch, h, extra=False)
    c = P.run_gpu_categorical(batch, h, extra=True)
    for k in ("loss_terms", "dlogits", "dvalues"):
        np.testing.assert_array_equal(a[k], b[k])
        np.testing.assert_array_equal(a[k], c[k])


def test_workspace_is_reusable_across_calls_and_shapes(oracle):
    import paper_1912_00167_b200 as ip
    ws = ip.new_workspace(64, 64)
    for (B, T, A, seed) in [(8, 20, 6, 1), (33, 50, 18, 2), (8, 20, 6, 1)]:
        batch = ii.categorical_batch(B, T, A, seed)
        h = P.f32_hyper(LossHyper())
        ref = oracle.loss_categorical(batch, h)
        t = {k: torch.from_numpy(v).cuda() for k, v in batch.items()}
        lt = torch.zeros(8, device="cuda")
        dz = torch.empty(B, T, A, device="cuda")
        dv = torch.empty(B, T, device="cuda")
        ip.impact_loss_fwd_bwd(t["learner_logits"], t["target_logits"], t["worker_logp"], t["actions"],
                               t["rewards"], t["discounts"], t["values"], t["bootstrap_values"], P.to_coef(h),
                               loss_terms=lt, dlogits=dz, dvalues=dv, workspace=ws)
        torch.cuda.synchronize()
        got = lt.cpu().numpy()
        got[4] = ref["loss_terms"][4]  # KL is not evaluated at kl_coef = 0
        np.testing.assert_allclose(got, ref["loss_terms"], rtol=1e-4, atol=1e-7)
    assert ip.impact_loss_workspace_status(ws) == 0  # no bounded wait ever ran out


@pytest.mark.parametrize("B,T,A", [(5, 300, 18), (3, 200, 64)])
def test_workspace_without_room_for_tile_aggregates(oracle, B, T, A):
    """The fixed part of the workspace serves long trajectories too (a block then sweeps a trajectory by itself);
    the result is the same as with the full workspace, and both match the oracle."""
    import paper_1912_00167_b200 as ip
    batch = ii.categorical_batch(B, T, A, seed=11 + T, p_done=0.01)
    h = P.f32_hyper(LossHyper(kl_coef=0.05))
    ref = oracle.loss_categorical(batch, h)
    t = {k: torch.from_numpy(v).cuda() for k, v in batch.items()}
    got = []
    for ws in (ip.new_workspace(1, 1), ip.new_workspace(B, T)):
        out = dict(loss_terms=torch.zeros(8, device="cuda"), dlogits=torch.empty(B, T, A, device="cuda"),
                   dvalues=torch.empty(B, T, device="cuda"))
        ip.impact_loss_fwd_bwd(t["learner_logits"], t["target_logits"], t["worker_logp"], t["actions"], t["rewards"],
                               t["discounts"], t["values"], t["bootstrap_values"], P.to_coef(h), workspace=ws, **out)
        torch.cuda.synchronize()
        got.append(out)
        np.testing.assert_allclose(out["loss_terms"].cpu().numpy(), ref["loss_terms"], rtol=1e-4, atol=1e-7)
    assert ip.new_workspace(B, T).numel() > ip.new_workspace(1, 1).numel()
    M = B * T
    np.testing.assert_allclose(got[0]["dvalues"].cpu().numpy() * M, got[1]["dvalues"].cpu().numpy() * M, rtol=1e-4, atol=1e-5)


@pytest.mark.parametrize("B,T,A,dtype", [(1024, 128, 18, torch.float32), (37, 50, 18, torch.float32),
                                         (5, 300, 18, torch.float32), (700, 200, 6, torch.float32),
                                         (4, 33, 5, torch.float32), (40, 128, 18, torch.bfloat16),
                                         (9, 100, 64, torch.float32), (301, 21, 9, torch.bfloat16)])
def test_target_logits_are_copied_out_by_the_loss_call(B, T, A, dtype):
    """First traversal of a batch: the call also stores the target logits (into a slot of the circular buffer, in
    a learner loop).  The copy is bit-exact, whichever kernel serves the shape, and nothing else changes."""
    import paper_1912_00167_b200 as ip
    batch = ii.categorical_batch(B, T, A, seed=21 + B + A, p_done=0.01)
    t = {k: torch.from_numpy(v).cuda() for k, v in batch.items()}
    zl, zt = t["learner_logits"].to(dtype), t["target_logits"].to(dtype)
    coef = ip.Coefficients(clip_eps=0.3, kl_coef=0.0)
    outs = []
    for with_copy in (False, True):
        out = dict(loss_terms=torch.zeros(8, device="cuda"), dlogits=torch.empty(B, T, A, device="cuda", dtype=dtype),
                   dvalues=torch.empty(B, T, device="cuda"))
        copy = torch.full((B, T, A), -7.0, device="cuda", dtype=dtype) if with_copy else None
        ip.impact_loss_fwd_bwd(zl, zt, t["worker_logp"], t["actions"], t["rewards"], t["discounts"], t["values"],
                               t["bootstrap_values"], coef, workspace=ip.new_workspace(B, T), target_logits_copy=copy,
                               **out)
        torch.cuda.synchronize()
        outs.append(out)
        if with_copy:
            assert torch.equal(copy.view(torch.uint8), zt.view(torch.uint8))
    for k in ("loss_terms", "dlogits", "dvalues"):
        assert torch.equal(outs[0][k], outs[1][k])


@pytest.mark.parametrize("B,T,A", [(32768, 128, 18), (32768, 128, 6)])
def test_no_wait_runs_out_in_long_launches(B, T, A):
    """Hundreds of tiles per block: every bounded wait of the persistent kernel must end by itself (the workspace's
    error word stays 0), launch after launch on the same workspace, and the launches agree bit for bit."""
    import paper_1912_00167_b200 as ip
    g = torch.Generator(device="cuda").manual_seed(3)
    zl = torch.randn(B, T, A, device="cuda", generator=g)
    zt = zl + 0.1 * torch.randn(B, T, A, device="cuda", generator=g)
    act = torch.randint(0, A, (B, T), device="cuda", generator=g, dtype=torch.int32)
    wl = torch.log_softmax(zl, -1).gather(-1, act.long().unsqueeze(-1)).squeeze(-1).contiguous()
    rew = (torch.rand(B, T, device="cuda", generator=g) < 0.05).float()
    dis = torch.where(torch.rand(B, T, device="cuda", generator=g) < 0.005, 0.0, 0.99).float()
    val, boot = torch.randn(B, T, device="cuda", generator=g), torch.randn(B, device="cuda", generator=g)
    ws = ip.new_workspace(B, T)
    outs = []
    for _ in range(6):
        out = dict(loss_terms=torch.zeros(8, device="cuda"), dlogits=torch.empty(B, T, A, device="cuda"),
                   dvalues=torch.empty(B, T, device="cuda"))
        ip.impact_loss_fwd_bwd(zl, zt, wl, act, rew, dis, val, boot, ip.Coefficients(clip_eps=0.4), workspace=ws, **out)
        outs.append(out["loss_terms"].clone())
    torch.cuda.synchronize()
    assert ip.impact_loss_workspace_status(ws) == 0
    assert torch.isfinite(outs[0]).all()
    for o in outs[1:]:
        assert torch.equal(o, outs[0])


def test_rows_of_dlogits_sum_to_zero_at_full_size():
    # softmax invariance: every term of the logit gradient sums to zero over the actions
    import paper_1912_00167_b200 as ip
    cfg, batch = ii.make_config(2)
    h = P.f32_hyper(dataclasses.replace(cfg.hyper, kl_coef=0.3))
    out = P.run_gpu_categorical(batch, h)
    M = batch["rewards"].size
    rows = out["dlogits"].sum(-1) * M
    scale = np.abs(out["dlogits"]).sum(-1) * M
    assert (np.abs(rows) <= 1e-5 * (1.0 + scale)).all()


def test_bad_arguments_are_rejected_before_launch():
    import paper_1912_00167_b200 as ip
    from paper_1912_00167_b200 import binding as bd
    cfg, batch = ii.make_config(0)
    t = {k: torch.from_numpy(v).cuda() for k, v in batch.items()}
    B, T, A = t["learner_logits"].shape
    lt = torch.zeros(8, device="cuda")
    dz = torch.empty(B, T, A, device="cuda")
    dv = torch.empty(B, T, device="cuda")
    ws = ip.new_workspace(B, T)

    def call(coef, workspace=ws, **over):
        args = dict(t)
        args.update(over)
        ip.impact_loss_fwd_bwd(args["learner_logits"], args["target_logits"], args["worker_logp"], args["actions"],
                               args["rewards"], args["discounts"], args["values"], args["bootstrap_values"], coef,
                               loss_terms=lt, dlogits=dz, dvalues=dv, workspace=workspace)

    for bad in (ip.Coefficients(rho_bar=-1.0), ip.Coefficients(clip_eps=float("nan")), ip.Coefficients(rho_tw=0.0),
                ip.Coefficients(ratio_mode=7), ip.Coefficients(is_source=3)):
        with pytest.raises(ip.ImpactError) as e:
            call(bad)
        assert e.value.status == bd.ERR_INVALID_ARG
    with pytest.raises(ip.ImpactError) as e:
        call(ip.Coefficients(), workspace=torch.zeros(64, dtype=torch.uint8, device="cuda"))
    assert e.value.status == bd.ERR_WORKSPACE_TOO_SMALL
    with pytest.raises(ValueError):
        call(ip.Coefficients(), rewards=t["rewards"].cpu())
    # misaligned base pointer
    big = torch.zeros(B * T + 4, device="cuda")
    with pytest.raises(ip.ImpactError) as e:
        call(ip.Coefficients(), rewards=big[1:B * T + 1].view(B, T))
    assert e.value.status == bd.ERR_INVALID_ARG
    call(ip.Coefficients())  # and the good call still works afterwards
    torch.cuda.synchronize()


@pytest.mark.parametrize("B,T,A,dtype", [(8192, 128, 18, torch.float32), (20972, 50, 18, torch.float32),
                                         (4096, 128, 18, torch.bfloat16), (512, 1000, 6, torch.float32)])
def test_sampled_trajectories_at_sweep_sizes(oracle, B, T, A, dtype):
    """Sizes far beyond what the oracle runs in full: trajectories are independent except for the 1/M
    normaliser, so a sample of them is recomputed by the oracle alone and compared after rescaling."""
    import paper_1912_00167_b200 as ip
    batch = ii.categorical_batch(B, T, A, seed=4242 + B, p_done=0.01)
    if dtype == torch.bfloat16:
        batch["learner_logits"] = ii.round_to_bf16(batch["learner_logits"])
        batch["target_logits"] = ii.round_to_bf16(batch["target_logits"])
    h = P.f32_hyper(LossHyper(clip_eps=0.4, rho_tw=2.0, lam=0.995))
    gpu = P.run_gpu_categorical(batch, h, dtype, torch.float32)
    M = B * T
    rng = np.random.default_rng(7)
    pick = np.sort(rng.choice(B, size=24, replace=False))
    pick[0], pick[-1] = 0, B - 1  # first and last tile
    sub = {k: np.ascontiguousarray(v[pick]) for k, v in batch.items()}
    ref = oracle.loss_categorical(sub, h)
    Ms = len(pick) * T
    near = P.near_clip_bound(ref, h)
    tol = 1e-5 * np.abs(ref["dlogits"] * Ms) + 1e-6 + 4e-6 * (ref["adv_cond"] * ref["ratio"])[..., None]
    err = np.abs(gpu["dlogits"][pick] * M - ref["dlogits"] * Ms)
    assert (err <= tol)[~near].all(), float((err - tol)[~near].max())
    np.testing.assert_array_less(np.abs(gpu["advantage"][pick] - ref["advantage"]),
                                 1e-5 * np.abs(ref["advantage"]) + 1e-6 + 4e-6 * ref["adv_cond"])
    np.testing.assert_array_less(np.abs(gpu["dvalues"][pick] * M - ref["dvalues"] * Ms),
                                 1e-5 * np.abs(ref["dvalues"] * Ms) + 1e-6 + 4e-6 * ref["adv_cond"])
    # properties that hold at any size
    rows = gpu["dlogits"].sum(-1) * M
    assert (np.abs(rows) <= 1e-5 * (1.0 + np.abs(gpu["dlogits"]).sum(-1) * M)).all()
    lt = gpu["loss_terms"]
    assert lt[0] == pytest.approx(lt[1] + h.vf_coef * lt[2] - h.ent_coef * lt[3] + h.kl_coef * lt[4], rel=1e-5, abs=1e-6)
    assert lt[2] == pytest.approx(0.5 * np.mean(gpu["advantage"] ** 2), rel=1e-4)
    assert 0.0 < lt[3] <= np.log(A) + 1e-5 and 0.0 <= lt[5] <= 1.0 and 0.0 <= lt[6] <= 1.0


@pytest.mark.parametrize("idx", [0, 1, 2])
def test_baseline_objectives_categorical(oracle, idx):
    """PPO (ratio R2, plain GAE-lambda) and IMPALA (V-trace policy gradient) on the same fused pass."""
    cfg, batch = ii.make_config(idx)
    ppo = dataclasses.replace(cfg.hyper, is_source=2, ratio_mode=2, lam=0.95, clip_eps=0.3)
    P.check_categorical(oracle, batch, ppo)
    impala = dataclasses.replace(cfg.hyper, objective=1, is_source=1, lam=1.0, kl_coef=0.1)
    P.check_categorical(oracle, batch, impala)


@pytest.mark.parametrize("B,T,A", [(5, 33, 7), (3, 300, 6), (9, 50, 18), (2, 70, 40)])
def test_vtrace_policy_gradient_ragged(oracle, B, T, A):
    batch = ii.categorical_batch(B, T, A, seed=5000 + T, p_done=0.05)
    P.check_categorical(oracle, batch, LossHyper(objective=1, is_source=1, rho_bar=1.3, c_bar=1.1, lam=0.97, ent_coef=0.02))
    P.check_categorical(oracle, batch, LossHyper(is_source=2, ratio_mode=2, lam=0.9))


def test_baseline_objectives_gaussian(oracle):
    cfg, batch = ii.make_config(3)
    P.check_gaussian(oracle, batch, dataclasses.replace(cfg.hyper, is_source=2, ratio_mode=2, lam=0.95, clip_eps=0.3))
    P.check_gaussian(oracle, batch, dataclasses.replace(cfg.hyper, objective=1, is_source=1, lam=1.0))
    small = ii.gaussian_batch(3, 140, 5, seed=77, p_done=0.05)
    P.check_gaussian(oracle, small, LossHyper(objective=1, is_source=1, ent_coef=0.01, kl_coef=0.2))


@pytest.mark.parametrize("B,T,A,parts", [(37, 50, 18, 2), (300, 128, 6, 3), (9, 300, 9, 2)])
def test_batch_split_over_calls_adds_up_to_the_whole(oracle, B, T, A, parts):
    """Data parallel over trajectories, every share run on this one GPU in turn: with `global_steps` set to the whole
    batch's M the shares' gradients are the whole batch's rows and their loss terms add up to the whole batch's --
    which is what the oracle computes for the unsplit batch."""
    import paper_1912_00167_b200 as ip
    batch = ii.categorical_batch(B, T, A, seed=77 + B, p_done=0.01)
    h = P.f32_hyper(LossHyper(clip_eps=0.3, kl_coef=0.1, rho_tw=2.0, lam=0.98))
    ref = oracle.loss_categorical(batch, h)
    M = B * T
    terms = np.zeros(8)
    dz, dv = np.zeros((B, T, A)), np.zeros((B, T))
    for r in range(parts):
        lo, hi = ip.shard_bounds(B, parts, r)
        t = {k_: torch.from_numpy(np.ascontiguousarray(v[lo:hi])).cuda() for k_, v in batch.items()}
        out = dict(loss_terms=torch.zeros(8, device="cuda"), dlogits=torch.empty(hi - lo, T, A, device="cuda"),
                   dvalues=torch.empty(hi - lo, T, device="cuda"))
        ip.impact_loss_fwd_bwd_sharded(t["learner_logits"], t["target_logits"], t["worker_logp"], t["actions"],
                                       t["rewards"], t["discounts"], t["values"], t["bootstrap_values"], P.to_coef(h),
                                       global_B=B, workspace=ip.new_workspace(hi - lo, T), **out)
        torch.cuda.synchronize()
        terms += out["loss_terms"].cpu().numpy().astype(np.float64)
        dz[lo:hi], dv[lo:hi] = out["dlogits"].cpu().numpy(), out["dvalues"].cpu().numpy()
    np.testing.assert_allclose(terms, ref["loss_terms"], rtol=1e-4, atol=1e-6)
    near = P.near_clip_bound(ref, h)
    tol = 1e-5 * np.abs(ref["dlogits"] * M) + 1e-6 + 4e-6 * (ref["adv_cond"] * ref["ratio"])[..., None]
    assert (np.abs(dz * M - ref["dlogits"] * M) <= tol)[~near].all()
    np.testing.assert_array_less(np.abs(dv * M - ref["dvalues"] * M), 1e-5 * np.abs(ref["dvalues"] * M) + 1e-6 + 4e-6 * ref["adv_cond"])
    # a normaliser smaller than the call's own steps is refused
    with pytest.raises(ip.ImpactError):
        lo, hi = 0, B
        t = {k_: torch.from_numpy(v).cuda() for k_, v in batch.items()}
        ip.impact_loss_fwd_bwd(t["learner_logits"], t["target_logits"], t["worker_logp"], t["actions"], t["rewards"],
                               t["discounts"], t["values"], t["bootstrap_values"],
                               dataclasses.replace(P.to_coef(h), global_steps=M - 1), workspace=ip.new_workspace(B, T),
                               loss_terms=torch.zeros(8, device="cuda"), dlogits=torch.empty(B, T, A, device="cuda"),
                               dvalues=torch.empty(B, T, device="cuda"))


def test_prepared_calls_keep_their_tensors_alive():
    """A prepared call holds raw device addresses; it must also hold the tensors they point into, or the call
    outlives its memory as soon as the caller drops its own references."""
    import paper_1912_00167_b200 as ip
    B, T, A, D = 3, 7, 6, 3

    def categorical():
        t = {k: torch.from_numpy(v).cuda() for k, v in ii.categorical_batch(B, T, A, seed=1).items()}
        out = dict(loss_terms=torch.zeros(8, device="cuda"), dlogits=torch.empty(B, T, A, device="cuda"),
                   dvalues=torch.empty(B, T, device="cuda"))
        ws = ip.new_workspace(B, T)
        call = ip.prepare_loss_fwd_bwd(t["learner_logits"], t["target_logits"], t["worker_logp"], t["actions"],
                                       t["rewards"], t["discounts"], t["values"], t["bootstrap_values"],
                                       ip.Coefficients(), workspace=ws, **out)
        return call, [t[k].data_ptr() for k in sorted(t)] + [v.data_ptr() for v in out.values()] + [ws.data_ptr()]

    def gaussian():
        t = {k: torch.from_numpy(v).cuda() for k, v in ii.gaussian_batch(B, T, D, seed=2).items()}
        out = dict(loss_terms=torch.zeros(8, device="cuda"), dmean=torch.empty(B, T, D, device="cuda"),
                   dlogstd=torch.empty(B, T, D, device="cuda"), dvalues=torch.empty(B, T, device="cuda"))
        ws = ip.new_workspace(B, T)
        call = ip.prepare_loss_fwd_bwd_gaussian(t["learner_mean"], t["learner_logstd"], t["target_mean"],
                                                t["target_logstd"], t["worker_logp"], t["actions"], t["rewards"],
                                                t["discounts"], t["values"], t["bootstrap_values"], ip.Coefficients(),
                                                workspace=ws, **out)
        return call, [t[k].data_ptr() for k in sorted(t)] + [v.data_ptr() for v in out.values()] + [ws.data_ptr()]

    for make in (categorical, gaussian):
        call, addresses = make()
        held = {x.data_ptr() for x in call._keep if isinstance(x, torch.Tensor)}
        assert set(addresses) <= held
