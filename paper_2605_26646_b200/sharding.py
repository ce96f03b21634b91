"""Host-side logic for running the path on several GPUs (one process per GPU).

The path shards by rollout group: a group's invocations and tokens stay on one rank, so the advantage
stage and the log-prob stage need no exchange.  The loss stage needs two small exchanges, both done here
with ``torch.distributed`` collectives (NCCL on GPUs, gloo in the CPU tests):

* before the step, the per-model valid-row counts are summed over ranks and passed to
  ``unity_ppo_loss_fwd_bwd`` as ``norm`` so that every rank scales its token terms by the global M_k;
* after the step, each dW_k is summed over ranks.  dHidden stays local.
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import torch
import torch.distributed as dist


def shard_groups(n_groups: int, rank: int, world: int) -> range:
    """Contiguous block of rollout groups owned by ``rank`` (sizes differ by at most one)."""
    base, extra = divmod(n_groups, world)
    start = rank * base + min(rank, extra)
    return range(start, start + base + (1 if rank < extra else 0))


def local_counts(tok_model: torch.Tensor, tok_mask: torch.Tensor, K: int) -> torch.Tensor:
    """Valid rows per model on this rank (float64 [K])."""
    return torch.bincount(tok_model[tok_mask != 0].long(), minlength=K).to(torch.float64)


def global_norm(counts: torch.Tensor, group=None) -> List[float]:
    """Sum the per-model counts over all ranks; returns max(M_k, 1) as python floats."""
    c = counts.clone()
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(c, group=group)
    return [max(float(x), 1.0) for x in c.tolist()]


def allreduce_grads(dW: Sequence[torch.Tensor], group=None) -> None:
    """Sum every dW_k over ranks, in place."""
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        for g in dW:
            dist.all_reduce(g, group=group)
