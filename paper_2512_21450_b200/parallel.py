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
    """Per-row weight 1 / (global number of valid tokens); the loss call multiplies it by the mask.
    Everything stays on the mask's device: the host never reads the count, so the step stays
    asynchronous.  (The loss call can also take the count itself: rl_loss_opts.token_count.)"""
    n = global_valid_count(mask, group)
    inv = torch.where(n > 0, 1.0 / n.clamp_min(1).to(torch.float64), torch.zeros_like(n, dtype=torch.float64))
    return inv.to(torch.float32).expand(mask.shape[0]).contiguous()


def allreduce_gradients(dW: torch.Tensor, loss: torch.Tensor, group=None):
    """Sum dW and the scalar loss over ranks in place (each rank's loss already uses global weights)."""
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(dW, op=dist.ReduceOp.SUM, group=group)
        dist.all_reduce(loss, op=dist.ReduceOp.SUM, group=group)
    return dW, loss


class SlabGradientReducer:
    """All-reduce of dW slab by slab while the backward pass is still running.

    The backward pass completes dW one slab of vocabulary rows at a time and reports each slab
    through the context's dW slab hook as soon as the launch that completes it has been enqueued.
    `on_slab` then records an event on the compute stream, makes a side stream wait for it and
    starts the all-reduce (sum) of exactly those rows there; the next slabs keep computing
    meanwhile.  `finish` makes the compute stream wait for the side stream (and reduces the scalar
    loss), after which dW holds the sum over ranks.  Slabs are reduced in the order they are
    reported, the same on every rank, so the collectives match up.  On CPU tensors (gloo) there
    are no streams and each slab is reduced at once; the result is the same.
    """

    def __init__(self, dW: torch.Tensor, group=None, single_rank_too: bool = False):
        self.dW = dW
        self.group = group
        self.min_world = 1 if single_rank_too else 2   # single_rank_too: run the collectives even in a group of one
        self.cuda = dW.is_cuda
        self.slabs = []
        self.world = dist.get_world_size(group) if dist.is_available() and dist.is_initialized() else 1
        if self.cuda:
            self.side = torch.cuda.Stream(device=dW.device)
            self.events = []

    def begin(self):
        """Call before the loss call of a step: the side stream must be done with the previous dW."""
        self.slabs = []
        if self.cuda:
            self.side.wait_stream(torch.cuda.current_stream(self.dW.device))

    def on_slab(self, slab: int, row_begin: int, row_end: int):
        self.slabs.append((slab, row_begin, row_end))
        if self.world < self.min_world:
            return
        rows = self.dW[row_begin:row_end]
        if not self.cuda:
            dist.all_reduce(rows, op=dist.ReduceOp.SUM, group=self.group)
            return
        k = len(self.slabs) - 1
        if k >= len(self.events):
            self.events.append(torch.cuda.Event())
        ev = self.events[k]
        ev.record(torch.cuda.current_stream(self.dW.device))
        self.side.wait_event(ev)
        with torch.cuda.stream(self.side):
            dist.all_reduce(rows, op=dist.ReduceOp.SUM, group=self.group)

    def finish(self, loss: torch.Tensor = None):
        """dW (and loss, if given) hold the sums over ranks for everything enqueued after this returns."""
        if self.cuda:
            torch.cuda.current_stream(self.dW.device).wait_stream(self.side)
        if loss is not None and self.world >= self.min_world:
            dist.all_reduce(loss, op=dist.ReduceOp.SUM, group=self.group)
        return self.dW


# ---------------------------------------------------------------------------------------------
# Vocabulary-parallel head: the rows of the LM-head weight are partitioned over the ranks of a
# group (rank r holds vocabulary ids [offsets[r], offsets[r+1])), every rank sees the same token
# rows.  Two exchanges are real: an all-gather of 16 bytes of softmax statistics per row and an
# all-reduce (sum) of the partial dH.  `compute` is the object that runs the three per-rank calls
# (a binding.Context on a GPU); it is a parameter so that the plumbing can be exercised on CPU
# ranks with a stand-in.
def shard_vocab(V: int, world: int, rank: int, multiple: int = 256):
    """Contiguous slice of the vocabulary for `rank`: (offset, size).  Slices are whole multiples of
    `multiple` rows (one tensor-core column tile) except the last, which takes the remainder."""
    tiles = -(-V // multiple)
    base, extra = divmod(tiles, world)
    start = (rank * base + min(rank, extra)) * multiple
    stop = ((rank + 1) * base + min(rank + 1, extra)) * multiple
    start, stop = min(start, V), min(stop, V)
    return start, stop - start


def vocab_parallel_logprobs(compute, H, W_shard, tokens, mask, vocab_offset, V_total, group=None):
    """(logp, entropy, lse) over the whole vocabulary, identical on every rank of the group."""
    stats = compute.rl_shard_logit_stats(H, W_shard, tokens, mask, vocab_offset, V_total)
    world = dist.get_world_size(group) if dist.is_available() and dist.is_initialized() else 1
    if world > 1:
        gathered = torch.empty((world,) + tuple(stats.shape), dtype=stats.dtype, device=stats.device)
        dist.all_gather(list(gathered.unbind(0)), stats.contiguous(), group=group)
    else:
        gathered = stats.reshape((1,) + tuple(stats.shape))
    return compute.rl_merge_logit_stats(gathered, mask)


def vocab_parallel_loss_fwd_bwd(compute, H, W_shard, tokens, old_logp, ref_logp, adv, mask, vocab_offset, V_total,
                                eps_low, eps_high, beta, group=None, **kw):
    """Forward and backward with the head split by vocabulary.  Returns dict(loss, dH, dW, logp,
    entropy): loss and dH (fp32, summed over the group) are the same on every rank; dW holds this
    rank's rows of the head gradient."""
    logp, ent, lse = vocab_parallel_logprobs(compute, H, W_shard, tokens, mask, vocab_offset, V_total, group)
    out = compute.rl_policy_loss_shard_bwd(H, W_shard, tokens, old_logp, ref_logp, adv, mask, vocab_offset, V_total,
                                           logp, ent, lse, eps_low, eps_high, beta, **kw)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(out["dH"], op=dist.ReduceOp.SUM, group=group)
    out["logp"], out["entropy"] = logp, ent
    return out
