"""Data-parallel plumbing for the LM-head loss path (one process per GPU, torch.distributed).

The path shards by prompts: token rows are independent in the forward pass and in dH, GRPO
groups stay whole on one rank, and dW is a sum over rows.  Two exchanges are real: the global
count of valid tokens (the token-mean weight is 1 / that count on every rank) and the sum of the
per-rank dW (and of the scalar loss).  Both are plain collectives on the default process group;
nothing here touches another GPU's memory directly.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def shard_prompts(n_prompts: int, world: int, rank: int):
    """Contiguous block of whole prompts (GRPO groups) for `rank`: (first_prompt, n_prompts_here)."""
    base, extra = divmod(n_prompts, world)
    start = rank * base + min(rank, extra)
    return start, base + (1 if rank < extra else 0)


def global_valid_count(mask: torch.Tensor, group=None) -> torch.Tensor:
    """Sum over ranks of the number of rows with mask != 0 (int64 tensor on mask's device)."""
    n = (mask != 0).sum().to(torch.int64).reshape(1)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(n, op=dist.ReduceOp.SUM, group=group)
    return n


def global_token_weight(mask: torch.Tensor, group=None) -> torch.Tensor:
    """Per-row weight 1 / (global number of valid tokens); the loss call multiplies it by the mask."""
    n = global_valid_count(mask, group)
    w = torch.zeros(mask.shape[0], dtype=torch.float32, device=mask.device)
    if int(n.item()) > 0:
        w.fill_(1.0 / float(n.item()))
    return w


def allreduce_gradients(dW: torch.Tensor, loss: torch.Tensor, group=None):
    """Sum dW and the scalar loss over ranks in place (each rank's loss already uses global weights)."""
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(dW, op=dist.ReduceOp.SUM, group=group)
        dist.all_reduce(loss, op=dist.ReduceOp.SUM, group=group)
    return dW, loss
