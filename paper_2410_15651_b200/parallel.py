"""Host-side logic for running the path data-parallel, one process per GPU.

The path shards by sequence with no exchange of logits: every row, and every sequence's GAE scan,
is independent.  The only coupling between ranks is the normaliser of the two losses, the number
of valid tokens N of the whole batch.  A rank that holds N_local of the N_global tokens calls
rlhf_ppo_loss_fwd_bwd on its shard with grad_scale multiplied by N_local / N_global (the call divides
by N_local itself), and the batch losses are the token-weighted means of the rank losses.  The
collectives are two scalar all-reduces; they work on any torch.distributed backend (NCCL on GPUs,
gloo on CPUs).
"""
from __future__ import annotations

from typing import Optional, Tuple

import torch
import torch.distributed as dist


def shard_range(n_sequences: int, world_size: int, rank: int) -> Tuple[int, int]:
    """Contiguous, balanced range [b0, b1) of the sequences that `rank` owns."""
    base, extra = divmod(n_sequences, world_size)
    b0 = rank * base + min(rank, extra)
    return b0, b0 + base + (1 if rank < extra else 0)


def token_counts(lengths_local: torch.Tensor, group=None) -> Tuple[int, int]:
    """(valid tokens on this rank, valid tokens on all ranks)."""
    n_local = lengths_local.to(torch.int64).sum().reshape(1)
    n_global = n_local.clone()
    if dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(n_global, op=dist.ReduceOp.SUM, group=group)
    return int(n_local.item()), int(n_global.item())


def grad_scale_for_global_mean(n_local: int, n_global: int, upstream: float = 1.0) -> float:
    """grad_scale to pass on this rank so that its gradients are those of the whole-batch token mean."""
    return upstream * n_local / n_global if n_global > 0 else 0.0


def combine_losses(loss_local: torch.Tensor, n_local: int, n_global: int, group=None) -> torch.Tensor:
    """Whole-batch [loss_pg, loss_vf] from the per-rank token means (float64, same on every rank)."""
    acc = loss_local.detach().to(torch.float64) * float(n_local)
    if dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(acc, op=dist.ReduceOp.SUM, group=group)
    return acc / float(n_global) if n_global > 0 else torch.zeros_like(acc)


def max_over_ranks(value: float, device: Optional[torch.device] = None, group=None) -> float:
    """Max of a host scalar over the ranks (used for device-timed milliseconds)."""
    t = torch.tensor([value], dtype=torch.float64, device=device)
    if dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    return float(t.item())


def sum_over_ranks(value: float, device: Optional[torch.device] = None, group=None) -> float:
    t = torch.tensor([value], dtype=torch.float64, device=device)
    if dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
    return float(t.item())
