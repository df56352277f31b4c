"""One train batch split over several GPUs (data parallel over trajectories).

Trajectories are independent: the only coupling between them is the 1/M normaliser of the
means (Algorithm 1) and the sums behind the eight loss terms.  So every rank runs the
fused loss on its own contiguous share of the B trajectories with `global_steps` set to the
whole batch's M -- its gradients are then final as they are -- and ONE collective remains:
the sum of the ranks' `loss_terms` (eight floats).  No kernel reads another GPU's memory.
"""
from __future__ import annotations

import dataclasses

import torch

from . import binding


def shard_bounds(B: int, world: int, rank: int) -> tuple[int, int]:
    """Trajectories [lo, hi) of rank `rank`: contiguous shares whose sizes differ by at most one."""
    if not (world >= 1 and 0 <= rank < world and B >= 0):
        raise ValueError("need world >= 1, 0 <= rank < world, B >= 0")
    base, extra = divmod(B, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def reduce_loss_terms(loss_terms: torch.Tensor, group=None) -> torch.Tensor:
    """Sums the ranks' loss terms in place (each rank's are sums over its steps divided by the global M)."""
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(loss_terms, op=dist.ReduceOp.SUM, group=group)
    return loss_terms


def impact_loss_fwd_bwd_sharded(learner_logits, target_logits, worker_logp, actions, rewards, discounts, values,
                                bootstrap_values, coef: binding.Coefficients, *, global_B: int, group=None,
                                loss_terms, dlogits, dvalues, vtarget=None, advantage=None, workspace,
                                stream=None) -> None:
    """`impact_loss_fwd_bwd` on this rank's trajectories of a batch of `global_B` trajectories in all.

    The tensors are the rank's share (B_local may differ between ranks, and may not be 0).  On return
    `dlogits` / `dvalues` are this share's rows of the whole batch's gradients and `loss_terms` holds the
    whole batch's terms on every rank.  The collective runs on the current stream of the process group's
    backend; with a non-default `stream` the caller orders the two."""
    T = learner_logits.shape[1]
    c = dataclasses.replace(coef, global_steps=int(global_B) * int(T))
    binding.impact_loss_fwd_bwd(learner_logits, target_logits, worker_logp, actions, rewards, discounts, values,
                                bootstrap_values, c, loss_terms=loss_terms, dlogits=dlogits, dvalues=dvalues,
                                vtarget=vtarget, advantage=advantage, workspace=workspace, stream=stream)
    reduce_loss_terms(loss_terms, group)
